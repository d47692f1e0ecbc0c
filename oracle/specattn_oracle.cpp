// SpecAttn verification hot path -- CPU ORACLE.
//
// TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct
// statement of what the hot path computes.  It shares no code, header, table
// or helper with the CUDA library and must never be called from the product
// path: only the tests, the smoke check and the benchmark's CPU-baseline leg
// may load it.
//
// What it states (paper passages in brackets):
//   O1  aggregate   a_bar[i] = sum over draft heads h and speculated queries s
//                   of A[h,s,i]                        [Sec. 3.4 item 1: one row
//                   a_{f(j)} per verifier layer; Alg. 1 "Sparse Attention Mask
//                   Creation": one token set per layer from the gamma maps]
//   O2  nucleus     the smallest largest-first prefix whose mass reaches
//                   p * sum(a_bar), ties at the threshold all kept
//                                                      [App. A Eq. 7; Alg. 2:
//                   target mass p*sum(a), membership test a_i >= theta]
//   O3  attention   softmax(q K^T / sqrt(d)) V restricted to the kept set
//                                                      [Eq. 1 restricted to the
//                   index set I of Eq. 2-3; normalised over I]
//
// Arithmetic: O1 is a chain of IEEE binary32 additions in a fixed order (this
// defines the aggregated value bit for bit); every mass in O2 and everything
// in O3 is binary64.  Compile WITHOUT fast-math and with -ffp-contract=off.
//
// Parity pins (tests/test_oracle_pins.py): worked rows with exact dyadic
// sums, brute-force subset enumeration, Alg. 2 bisection run to convergence,
// closed forms, monotonicity / permutation / scaling invariants for O2; a
// dense fp64 library softmax-attention, single-token, zero-key and LSE-merge
// identities and the App. A error bound for O3; an order-sensitive fp32 sum
// for O1.  No function here is "parity unpinned".

#include <algorithm>
#include <cfloat>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>

#if defined(_OPENMP)
#include <omp.h>
#endif

namespace {

inline double bf16_bits_to_double(uint16_t h) {
  uint32_t u = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &u, sizeof(f));
  return static_cast<double>(f);
}

// A probability is valid when it is a finite number >= 0 (-0.0 counts as 0).
inline bool valid_prob(float x) { return (x >= 0.0f) && (x <= FLT_MAX); }

}  // namespace

extern "C" {

enum {
  ORACLE_OK = 0,
  ORACLE_INVALID_PROB = 1,
  ORACLE_OVERFLOW = 2,
};

int specattn_oracle_num_threads(void) {
#if defined(_OPENMP)
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// ---------------------------------------------------------------------------
// O1.  Aggregated draft attention row for one (draft layer, sequence, group).
//   A          [n_heads, gamma, L_stride] binary32, position contiguous
//   head_group NULL: every head feeds the row; else only heads with
//              head_group[h] == g
//   a_bar      [L] output
// Order of the binary32 additions: start from +0, heads ascending, inside a
// head the speculated queries ascending.  Returns ORACLE_INVALID_PROB if any
// contributing input is negative, NaN or infinite, or if the binary32 chain
// itself overflows (impossible for probabilities) -- the row is still written.
// [Sec. 3.4 item 1; Alg. 1 "Sparse Attention Mask Creation"]
// ---------------------------------------------------------------------------
int specattn_oracle_aggregate(const float* A, int n_heads, int gamma, int64_t L_stride, int L,
                              const int32_t* head_group, int g, float* a_bar) {
  int status = ORACLE_OK;
  for (int i = 0; i < L; ++i) {
    float acc = 0.0f;
    for (int h = 0; h < n_heads; ++h) {
      if (head_group != nullptr && head_group[h] != g) continue;
      for (int s = 0; s < gamma; ++s) {
        const float x = A[(static_cast<int64_t>(h) * gamma + s) * L_stride + i];
        if (!valid_prob(x)) status = ORACLE_INVALID_PROB;
        acc = acc + x;
      }
    }
    if (!(acc <= FLT_MAX)) status = ORACLE_INVALID_PROB;  // the binary32 chain overflowed
    a_bar[i] = acc;
  }
  return status;
}

// ---------------------------------------------------------------------------
// O2.  Top-p nucleus of one non-negative row by explicit full sort.
//   total  = sum_i (double) a[i], index order
//   p >= 1: every position is kept (a rule, not arithmetic)
//   else    target = (double) p * total; positions sorted by value descending
//           (index ascending among equals); C_k = running binary64 sum in that
//           order; k* = min{k : C_k >= target}; theta = value of the k*-th;
//           kept = {i : a[i] >= theta}, emitted in ascending position.
//   diag[0..5] = total, target, M_gt (mass strictly above theta),
//                M_ge (mass of the kept set), margin, theta
//   margin = min(M_ge - target, target - M_gt) / total  (1 when total == 0 or
//            p >= 1): how far the decision is from flipping.
// Writes at most idx_cap positions; returns the true kept count.
// [App. A Eq. 7; Alg. 2 lines "M_target <- p * sum a" and "T_s <- {i: a_i >= theta}"]
// ---------------------------------------------------------------------------
int64_t specattn_oracle_nucleus(const float* a, int L, float p, int32_t* idx, int64_t idx_cap,
                                double* diag) {
  double total = 0.0;
  for (int i = 0; i < L; ++i) total += static_cast<double>(a[i]);
  double target = static_cast<double>(p) * total;
  double m_gt = 0.0, m_ge = total, margin = 1.0, theta = 0.0;
  int64_t count = 0;

  if (L > 0 && !(p >= 1.0f)) {
    std::vector<int32_t> order(L);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(),
                     [a](int32_t x, int32_t y) { return a[x] > a[y]; });
    double c = 0.0;
    int k_star = L;  // 1-based length of the prefix
    std::vector<double> prefix(L);
    for (int k = 0; k < L; ++k) {
      c += static_cast<double>(a[order[k]]);
      prefix[k] = c;
      if (c >= target) {
        k_star = k + 1;
        break;
      }
    }
    const float th = a[order[k_star - 1]];
    theta = static_cast<double>(th);
    // first position of the tie group in sorted order
    int first = k_star - 1;
    while (first > 0 && a[order[first - 1]] == th) --first;
    m_gt = (first > 0) ? prefix[first - 1] : 0.0;
    // extend the running sum to the end of the tie group
    int last = k_star;  // exclusive
    double cg = prefix[k_star - 1];
    while (last < L && a[order[last]] == th) {
      cg += static_cast<double>(a[order[last]]);
      ++last;
    }
    m_ge = cg;
    margin = (total > 0.0) ? std::min(m_ge - target, target - m_gt) / total : 1.0;
    for (int i = 0; i < L; ++i) {
      if (a[i] >= th) {
        if (count < idx_cap) idx[count] = i;
        ++count;
      }
    }
  } else {
    for (int i = 0; i < L; ++i) {
      if (count < idx_cap) idx[count] = i;
      ++count;
    }
    theta = 0.0;
  }
  if (diag != nullptr) {
    diag[0] = total;
    diag[1] = target;
    diag[2] = m_gt;
    diag[3] = m_ge;
    diag[4] = margin;
    diag[5] = theta;
  }
  return count;
}

// ---------------------------------------------------------------------------
// O1 + O2 over a whole step: every draft layer that some target layer maps to,
// every sequence, every group.
//   draft_probs[u]  [B, n_heads, gamma, L_stride] binary32 (NULL allowed for
//                   draft layers no target layer maps to)
//   layer_map       [n_target_layers] in [-1, n_draft_layers); -1 = dense layer
//   idx             [n_draft_layers, B, G, idx_stride]   ascending positions
//   counts, status  [n_draft_layers, B, G]
//   diag            [n_draft_layers, B, G, 6] or NULL (see specattn_oracle_nucleus)
// A row with an invalid probability gets status INVALID_PROB and count 0.  A
// list longer than idx_stride is cut to its first idx_stride positions, keeps
// its true count and gets OVERFLOW.  Lists of unmapped draft layers are left
// untouched.                                  [Alg. 1 lines "i* <- f(j)", "T_j <- ..."]
// ---------------------------------------------------------------------------
void specattn_oracle_select_topp(const float* const* draft_probs, int n_draft_layers,
                                 const int32_t* layer_map, int n_target_layers, int B, int n_heads,
                                 int gamma, int G, int64_t L_stride, const int32_t* kv_len,
                                 const int32_t* head_group, float p, int32_t* idx,
                                 int64_t idx_stride, int32_t* counts, int32_t* status,
                                 double* diag) {
  std::vector<char> used(n_draft_layers, 0);
  for (int j = 0; j < n_target_layers; ++j)
    if (layer_map[j] >= 0 && layer_map[j] < n_draft_layers) used[layer_map[j]] = 1;
  const int64_t n_lists = static_cast<int64_t>(n_draft_layers) * B * G;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t li = 0; li < n_lists; ++li) {
    const int u = static_cast<int>(li / (static_cast<int64_t>(B) * G));
    const int b = static_cast<int>((li / G) % B);
    const int g = static_cast<int>(li % G);
    if (!used[u]) continue;
    const int L = kv_len[b];
    std::vector<float> a_bar(std::max(L, 1));
    const float* A = draft_probs[u] + static_cast<int64_t>(b) * n_heads * gamma * L_stride;
    int st = specattn_oracle_aggregate(A, n_heads, gamma, L_stride, L, head_group, g,
                                       a_bar.data());
    double* dg = diag ? diag + li * 6 : nullptr;
    if (st == ORACLE_INVALID_PROB) {
      counts[li] = 0;
      status[li] = ORACLE_INVALID_PROB;
      if (dg) for (int k = 0; k < 6; ++k) dg[k] = std::numeric_limits<double>::quiet_NaN();
      continue;
    }
    int64_t c = specattn_oracle_nucleus(a_bar.data(), L, p, idx + li * idx_stride, idx_stride, dg);
    counts[li] = static_cast<int32_t>(c);
    status[li] = (c > idx_stride) ? ORACLE_OVERFLOW : ORACLE_OK;
  }
}

// ---------------------------------------------------------------------------
// O2b.  The bisection of Alg. 2 for one row, taken literally, with a fixed number of
// iterations (the paper's implementation note: 10).
//   total  = sum_i (double) a[i], index order; target = (double) p * total
//   theta_high = max_i a[i], theta_low = 0          (binary32)
//   repeat n_iters times:
//     theta_mid = (theta_high + theta_low) / 2      (binary32)
//     M_current = sum_{i : a[i] >= theta_mid} (double) a[i], index order
//     M_current < target ? theta_high = theta_mid : theta_low = theta_mid
//   kept = {i : a[i] >= theta_mid of the last iteration}, ascending.
// Unlike O2 the result may fall short of the target mass (when the last midpoint lies above the
// exact threshold) or keep more than the smallest set (when it lies below).
//   p >= 1: every position is kept (the same rule as O2).  n_iters >= 1.
//   diag[0..5] = total, target, mass of the kept set, theta_mid (last), margin, max
//   margin = min over the iterations of |M_current - target| / total (1 when total == 0 or
//            p >= 1): how far the nearest comparison was from flipping.
// [Alg. 2, the loop over theta and "T_s <- {i : a_{s,i} >= theta_mid}"; footnote to Sec. 3.4]
// ---------------------------------------------------------------------------
int64_t specattn_oracle_bisect(const float* a, int L, float p, int n_iters, int32_t* idx,
                               int64_t idx_cap, double* diag) {
  double total = 0.0;
  float vmax = 0.0f;
  for (int i = 0; i < L; ++i) {
    total += static_cast<double>(a[i]);
    if (a[i] > vmax) vmax = a[i];
  }
  const double target = static_cast<double>(p) * total;
  double margin = 1.0, kept_mass = total;
  float theta_mid = 0.0f;
  int64_t count = 0;
  if (L > 0 && !(p >= 1.0f)) {
    float theta_high = vmax, theta_low = 0.0f;
    for (int it = 0; it < n_iters; ++it) {
      theta_mid = (theta_high + theta_low) / 2.0f;
      double m_current = 0.0;
      for (int i = 0; i < L; ++i)
        if (a[i] >= theta_mid) m_current += static_cast<double>(a[i]);
      if (total > 0.0) margin = std::min(margin, std::fabs(m_current - target) / total);
      if (m_current < target) theta_high = theta_mid; else theta_low = theta_mid;
      kept_mass = m_current;
    }
  }
  for (int i = 0; i < L; ++i) {
    if (a[i] >= theta_mid) {
      if (count < idx_cap) idx[count] = i;
      ++count;
    }
  }
  if (diag != nullptr) {
    diag[0] = total;
    diag[1] = target;
    diag[2] = kept_mass;
    diag[3] = static_cast<double>(theta_mid);
    diag[4] = margin;
    diag[5] = static_cast<double>(vmax);
  }
  return count;
}

// ---------------------------------------------------------------------------
// O1 + O2 over a whole step with the selection variants of Alg. 2.
//   per_step == 0: one row per list, aggregated over heads AND speculated queries (O1), one
//                  nucleus -- specattn_oracle_select_topp when n_iters == 0.
//   per_step == 1: Alg. 2 as printed: for every speculated query s the row
//                  a_s[i] = sum over the group's heads h (ascending, binary32, from +0) of
//                  A[h, s, i] gets its own nucleus T_s, and the list is the union of the T_s.
//   n_iters == 0: exact nucleus (O2); n_iters >= 1: literal bisection (O2b).
//   chunk > 1:    selection at chunk granularity (Sec. 4: "chunk size ... 16"): the row that
//                 is searched holds one score per chunk of `chunk` consecutive positions, the
//                 binary32 sum of the chunk's values in ascending order; kept chunks keep all
//                 their positions.  chunk == 1 is per-position selection.
// Other arguments, truncation and status as in specattn_oracle_select_topp.
//   diag [n_draft_layers, B, G, 6]: [4] = smallest margin over the rows of the list, the other
//   entries are those of the last row processed.
// [Alg. 2 "for s = 1 to gamma ... T <- T u T_s"]
// ---------------------------------------------------------------------------
void specattn_oracle_select_variant(const float* const* draft_probs, int n_draft_layers,
                                    const int32_t* layer_map, int n_target_layers, int B,
                                    int n_heads, int gamma, int G, int64_t L_stride,
                                    const int32_t* kv_len, const int32_t* head_group, float p,
                                    int per_step, int n_iters, int chunk, int32_t* idx,
                                    int64_t idx_stride, int32_t* counts, int32_t* status,
                                    double* diag) {
  std::vector<char> used(n_draft_layers, 0);
  for (int j = 0; j < n_target_layers; ++j)
    if (layer_map[j] >= 0 && layer_map[j] < n_draft_layers) used[layer_map[j]] = 1;
  const int64_t n_lists = static_cast<int64_t>(n_draft_layers) * B * G;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t li = 0; li < n_lists; ++li) {
    const int u = static_cast<int>(li / (static_cast<int64_t>(B) * G));
    const int b = static_cast<int>((li / G) % B);
    const int g = static_cast<int>(li % G);
    if (!used[u]) continue;
    const int L = kv_len[b];
    const float* A = draft_probs[u] + static_cast<int64_t>(b) * n_heads * gamma * L_stride;
    std::vector<float> row(std::max(L, 1));
    std::vector<int32_t> tmp(std::max(L, 1));
    std::vector<float> score(std::max(L, 1));
    std::vector<char> in_set(std::max(L, 1), 0);
    double dg[6] = {0, 0, 0, 0, 1.0, 0};
    double min_margin = 1.0;
    bool invalid = false;
    const int n_rows = per_step ? gamma : 1;
    for (int s = 0; s < n_rows && !invalid; ++s) {
      int st;
      if (per_step) {
        // heads only: the row of speculated query s
        st = ORACLE_OK;
        for (int i = 0; i < L; ++i) {
          float acc = 0.0f;
          for (int h = 0; h < n_heads; ++h) {
            if (head_group != nullptr && head_group[h] != g) continue;
            const float x = A[(static_cast<int64_t>(h) * gamma + s) * L_stride + i];
            if (!valid_prob(x)) st = ORACLE_INVALID_PROB;
            acc = acc + x;
          }
          if (!(acc <= FLT_MAX)) st = ORACLE_INVALID_PROB;
          row[i] = acc;
        }
      } else {
        st = specattn_oracle_aggregate(A, n_heads, gamma, L_stride, L, head_group, g, row.data());
      }
      if (st == ORACLE_INVALID_PROB) {
        invalid = true;
        break;
      }
      // chunk > 1: the selection runs over chunk scores, score_j = +0 + a[j*chunk] + a[j*chunk+1]
      // + ... (binary32, ascending, the last chunk cut at L), and a kept chunk keeps all its
      // positions
      const int n_sel = (chunk > 1) ? (L + chunk - 1) / chunk : L;
      if (chunk > 1) {
        for (int j = 0; j < n_sel; ++j) {
          float acc = 0.0f;
          for (int i = j * chunk; i < std::min(L, (j + 1) * chunk); ++i) acc = acc + row[i];
          if (!(acc <= FLT_MAX)) invalid = true;
          score[j] = acc;
        }
        if (invalid) break;
      }
      const float* sel = (chunk > 1) ? score.data() : row.data();
      const int64_t c = (n_iters > 0)
                            ? specattn_oracle_bisect(sel, n_sel, p, n_iters, tmp.data(), n_sel, dg)
                            : specattn_oracle_nucleus(sel, n_sel, p, tmp.data(), n_sel, dg);
      min_margin = std::min(min_margin, dg[4]);
      for (int64_t k = 0; k < c; ++k) {
        if (chunk > 1) {
          for (int i = tmp[k] * chunk; i < std::min(L, (tmp[k] + 1) * chunk); ++i) in_set[i] = 1;
        } else {
          in_set[tmp[k]] = 1;
        }
      }
    }
    // (an invalid probability in any contributing row voids the list: the loop stopped there)
    double* out_dg = diag ? diag + li * 6 : nullptr;
    if (invalid) {
      counts[li] = 0;
      status[li] = ORACLE_INVALID_PROB;
      if (out_dg) for (int k = 0; k < 6; ++k) out_dg[k] = std::numeric_limits<double>::quiet_NaN();
      continue;
    }
    int64_t c = 0;
    int32_t* out = idx + li * idx_stride;
    for (int i = 0; i < L; ++i)
      if (in_set[i]) {
        if (c < idx_stride) out[c] = i;
        ++c;
      }
    counts[li] = static_cast<int32_t>(c);
    status[li] = (c > idx_stride) ? ORACLE_OVERFLOW : ORACLE_OK;
    if (out_dg) {
      for (int k = 0; k < 6; ++k) out_dg[k] = dg[k];
      out_dg[4] = min_margin;
    }
  }
}

// ---------------------------------------------------------------------------
// O3 core.  Softmax attention of M query rows over c gathered key/value rows.
//   q  [M, d] bf16 bits, K and V [c, d] bf16 bits (row stride given in elements)
//   s_i = (q . k_i) * scale ; m = max_i s_i ; l = sum_i exp(s_i - m)
//   out[r, :] = sum_i exp(s_i - m) v_i / l ;  lse[r] = m + ln l   (natural log)
//   c == 0: out = 0, lse = -inf.
// [Eq. 1, restricted to the selected set I of Eq. 2-3 and normalised over I]
// ---------------------------------------------------------------------------
void specattn_oracle_attend_rows(const uint16_t* q, int64_t q_stride, const uint16_t* K,
                                 int64_t k_stride, const uint16_t* V, int64_t v_stride, int M,
                                 int64_t c, int d, double scale, double* out, double* lse) {
  std::vector<double> s(std::max<int64_t>(c, 1));
  for (int r = 0; r < M; ++r) {
    double* o = out + static_cast<int64_t>(r) * d;
    for (int e = 0; e < d; ++e) o[e] = 0.0;
    if (c == 0) {
      lse[r] = -std::numeric_limits<double>::infinity();
      continue;
    }
    double m = -std::numeric_limits<double>::infinity();
    for (int64_t i = 0; i < c; ++i) {
      double dot = 0.0;
      for (int e = 0; e < d; ++e)
        dot += bf16_bits_to_double(q[r * q_stride + e]) * bf16_bits_to_double(K[i * k_stride + e]);
      s[i] = dot * scale;
      m = std::max(m, s[i]);
    }
    double l = 0.0;
    for (int64_t i = 0; i < c; ++i) l += std::exp(s[i] - m);
    for (int64_t i = 0; i < c; ++i) {
      const double w = std::exp(s[i] - m) / l;
      for (int e = 0; e < d; ++e) o[e] += w * bf16_bits_to_double(V[i * v_stride + e]);
    }
    lse[r] = m + std::log(l);
  }
}

// ---------------------------------------------------------------------------
// O3 over one target layer of a paged cache.
//   q          [B, T, H_q, d] bf16 bits
//   kv_pages   bf16 bits; element (page, kv, slot, head, e) at
//              page*stride_page + kv*stride_kv + slot*stride_slot + head*stride_head + e
//              (kv = 0 keys, 1 values)
//   block_table[b*bt_stride + i/page_size] = page of position i; NULL = the
//              cache is contiguous: position i of sequence b is at page
//              b*ceil(max_len/page_size)+i/page_size with max_len = bt_stride
//              (bt_stride is then read as "pages per sequence")
//   idx/counts the lists of ONE draft layer: [B, G, idx_stride], [B, G];
//              dense != 0: every position < kv_len[b] is attended, lists unread
//   query head h uses kv head h / (H_q/H_kv) and list g = (G == 1 ? 0 : kv head)
//   tail_len   the in-flight tokens: positions kv_len[b] + j, j < tail_len, already in the
//              cache; query t additionally attends those with j <= t + (tail_len - T), i.e.
//              causally among the tokens being verified (tail_len = T: token t sees itself)
//   out [B, T, H_q, d] and lse [B, T, H_q] binary64.
// All T queries and all heads of a group share one list.
// [Alg. 1 "Verification with Sparse Attention": one mask per layer for the
//  gamma+1 verifier predictions; Eq. 1-3]
// ---------------------------------------------------------------------------
void specattn_oracle_sparse_verify(int B, int T, int Hq, int Hkv, int d, int page_size, int G,
                                   const uint16_t* q, const uint16_t* kv_pages, int64_t stride_page,
                                   int64_t stride_kv, int64_t stride_slot, int64_t stride_head,
                                   const int32_t* block_table, int64_t bt_stride,
                                   const int32_t* kv_len, const int32_t* idx, int64_t idx_stride,
                                   const int32_t* counts, int dense, double scale, int tail_len,
                                   double* out, double* lse) {
  const int grp = Hq / Hkv;
  if (scale == 0.0) scale = 1.0 / std::sqrt(static_cast<double>(d));
  const int64_t n_units = static_cast<int64_t>(B) * Hkv;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t unit = 0; unit < n_units; ++unit) {
    const int b = static_cast<int>(unit / Hkv);
    const int hk = static_cast<int>(unit % Hkv);
    const int g = (G == 1) ? 0 : hk;
    const int64_t li = static_cast<int64_t>(b) * G + g;
    const int64_t c = dense ? kv_len[b] : std::min<int64_t>(counts[li], idx_stride);
    const int64_t ct = c + tail_len;  // listed rows first, then the in-flight tokens
    std::vector<uint16_t> Kr(std::max<int64_t>(ct, 1) * d), Vr(std::max<int64_t>(ct, 1) * d);
    for (int64_t k = 0; k < ct; ++k) {
      const int64_t pos = (k >= c) ? (kv_len[b] + (k - c)) : (dense ? k : idx[li * idx_stride + k]);
      const int64_t logical_page = pos / page_size;
      const int64_t page = block_table ? block_table[b * bt_stride + logical_page]
                                       : b * bt_stride + logical_page;
      const int64_t slot = pos % page_size;
      const uint16_t* base = kv_pages + page * stride_page + slot * stride_slot + hk * stride_head;
      std::memcpy(&Kr[k * d], base, sizeof(uint16_t) * d);
      std::memcpy(&Vr[k * d], base + stride_kv, sizeof(uint16_t) * d);
    }
    for (int t = 0; t < T; ++t) {
      // query t sees the whole list and the first (t + tail_len - T + 1) in-flight tokens
      int64_t n_tail = static_cast<int64_t>(t) + tail_len - T + 1;
      n_tail = std::max<int64_t>(0, std::min<int64_t>(n_tail, tail_len));
      for (int hh = 0; hh < grp; ++hh) {
        const int h = hk * grp + hh;
        const int64_t row = (static_cast<int64_t>(b) * T + t) * Hq + h;
        specattn_oracle_attend_rows(q + row * d, d, Kr.data(), d, Vr.data(), d, 1, c + n_tail, d, scale,
                                    out + row * d, lse + row);
      }
    }
  }
}

}  // extern "C"
