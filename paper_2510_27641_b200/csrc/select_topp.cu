// specattn_select_topp: aggregation of draft attention rows, exact sorting-free top-p
// threshold search and ordered compaction, for sm_100a.
//
// Paper: Sec. 3.4 / Alg. 2 (target mass p * sum a, membership a_i >= theta) and App. A Eq. 7
// (smallest set reaching mass p).  Alg. 2 bisects theta in the probability domain with one
// full pass over the row per iteration; here the same fixed point is reached exactly in three
// radix passes over the binary32 bit pattern (11 + 10 + 10 bits), each pass building a
// histogram of (count, mass) per bin, and the row never leaves the chip between passes.
//
// Mapping to the GPU: one thread-block cluster (1, 2, 4 or 8 CTAs) per index list.  Each CTA
//   1. streams its slice of positions of all contributing (head, query) rows from HBM in 8 KB
//      row pieces: every thread copies the two float4 columns it will add itself with 16-byte
//      cp.async into its own shared-memory ring slots, eight pieces ahead (64 KB in flight per
//      CTA, no registers held, no barrier needed), adds them in the fixed order that defines
//      the aggregated row and keeps the aggregated slice in shared memory (it is never written
//      to global memory).  (A 1-D bulk-copy ring fed by a producer warp was measured first:
//      like the gather in the verify kernel it stalled near 25 GB/s per SM.)
//   2. builds the level histogram in shared memory (64-bit packed count|mantissa-sum atomics;
//      all values of a bin share one exponent, so the mantissa sum is an exact integer and
//      the result does not depend on the order of the atomics);
//   3. the cluster reduces the histograms through distributed shared memory, every CTA scans
//      the reduced bins in binary64 in one fixed order and all arrive at the same bin;
//   4. after three levels the threshold is known bit-exactly; each CTA compacts its kept
//      positions in ascending order behind the counts of the lower-ranked CTAs.
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <float.h>
#include <stdint.h>
#include <string.h>

#include <atomic>

#include "ptx.cuh"
#include "specattn.h"

namespace cg = cooperative_groups;

namespace specattn {

extern std::atomic<long long> g_launch_count;

namespace {

constexpr int kThreads = 256;            // worker threads
constexpr int kWarps = kThreads / 32;
constexpr int kBlock = kThreads;
constexpr int kChunk = 2048;             // positions per staged row piece (8 KB)
constexpr int kDepth = 8;                // row pieces in flight per thread (ring of 8 x 8 KB)
constexpr int kL1Bins = 2048;        // sign(0) + 8 exponent bits + 3 mantissa bits
constexpr int kL23Bins = 1024;       // 10 mantissa bits per later level
constexpr int kHistSlots = kL1Bins + 8;  // slot kL1Bins counts invalid inputs, the next one timeouts
constexpr int kInvalidSlot = kL1Bins;
constexpr int kTimeoutSlot = kL1Bins + 1;
constexpr int kGroup = 32;           // bins per scan group
constexpr int kMaxGroups = kL1Bins / kGroup;
constexpr int kSliceCap = 32768;     // positions per CTA
constexpr unsigned long long kOne = 1ull << 44;  // count field of a packed bin
constexpr unsigned long long kMantMask = kOne - 1;

struct SelectParams {
  const float* probs[SPECATTN_MAX_DRAFT_LAYERS];  // per used slot
  int layer_of[SPECATTN_MAX_DRAFT_LAYERS];        // draft layer id of a used slot
  signed char head_group[SPECATTN_MAX_DRAFT_HEADS];
  int has_groups;
  int n_used, B, H, gamma, G;
  long long L_stride;
  const int* kv_len;
  float p;
  int keep_all;
  int* idx;
  long long idx_stride;
  int* counts;
  int* status;
  double* diag;
};

struct Shared {
  unsigned long long hist[kHistSlots];
  double* mass;        // [kL1Bins] reduced bin masses  } both alias the staging ring, which is
  unsigned int* cnt;   // [kL1Bins] reduced bin counts  } idle once the slice is aggregated
  long long row_off[SPECATTN_MAX_ROWS_PER_LIST];  // element offset of each contributing row, in add order
  double grp_mass[kMaxGroups];
  double suf_mass[kMaxGroups + 1];
  unsigned int grp_cnt[kMaxGroups];
  unsigned int suf_cnt[kMaxGroups + 1];
  int warp_cnt[kWarps];
  int n_rows;
  int found_group;
  int found_bin;
  unsigned int cnt_above;   // elements in bins strictly above the found bin (incl. carry)
  unsigned int cnt_bin;     // elements in the found bin
  double mass_above;        // mass strictly above the found bin (incl. carry)
  double mass_ge;           // mass_above + mass of the found bin
  int local_kept;           // read by the other CTAs of the cluster
};

__device__ __forceinline__ double pow2_double(int k) {  // 2^k, k in the normal range
  return __longlong_as_double(static_cast<long long>(k + 1023) << 52);
}

// Adds one aggregated value to a histogram bin.  When the whole warp hits the same bin the
// packed values are summed with shuffles and one lane issues the atomic.
__device__ __forceinline__ void hist_add(unsigned long long* hist, bool take, int bin,
                                         unsigned int mant) {
  const unsigned full = 0xffffffffu;
  const unsigned takers = __ballot_sync(full, take);
  if (takers == 0) return;
  const int leader = __ffs(takers) - 1;
  const int lead_bin = __shfl_sync(full, bin, leader);
  const bool same = __all_sync(full, !take || bin == lead_bin);
  if (same && __popc(takers) > 4) {
    unsigned int m = take ? mant : 0u;
    unsigned long long v = take ? (kOne | m) : 0ull;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(full, v, o);
    if ((threadIdx.x & 31) == leader) atomicAdd(&hist[lead_bin], v);
  } else if (take) {
    atomicAdd(&hist[bin], kOne | mant);
  }
}

__device__ __forceinline__ unsigned int mantissa_of(unsigned int key) {
  return (key >> 23) ? ((key & 0x7fffffu) | 0x800000u) : (key & 0x7fffffu);
}

// Cluster-wide reduction of the per-CTA histograms into (cnt, mass) for `nbins` bins, the
// result replicated in every CTA.  `exp_of_bin(bin)` gives the binary exponent that scales the
// integer mantissa sum of that bin.
template <typename ExpFn>
__device__ void reduce_hist(cg::cluster_group& cluster, Shared& sh, int nbins, ExpFn exp_of_bin) {
  const unsigned cs = cluster.num_blocks();
  const unsigned rank = cluster.block_rank();
  const int per = nbins / static_cast<int>(cs);
  double* const mass = sh.mass;
  unsigned int* const cnt = sh.cnt;
  cluster.sync();  // every CTA's histogram is complete
  const int lo = static_cast<int>(rank) * per;
  for (int bin = lo + threadIdx.x; bin < lo + per && threadIdx.x < kThreads; bin += kThreads) {
    unsigned long long s = 0;
    for (unsigned r = 0; r < cs; ++r) s += *cluster.map_shared_rank(&sh.hist[bin], r);
    cnt[bin] = static_cast<unsigned int>(s >> 44);
    mass[bin] = static_cast<double>(s & kMantMask) * pow2_double(exp_of_bin(bin));
  }
  cluster.sync();  // every owner's part is reduced; remote histograms are no longer read
  for (int bin = threadIdx.x; bin < nbins && threadIdx.x < kThreads; bin += kThreads) {
    const unsigned owner = static_cast<unsigned>(bin / per);
    if (owner != rank) {
      cnt[bin] = *cluster.map_shared_rank(&cnt[bin], owner);
      mass[bin] = *cluster.map_shared_rank(&mass[bin], owner);
    }
  }
  __syncthreads();
}

// Finds the highest bin at which the mass accumulated from the top (starting from
// `carry_mass` / `carry_cnt` already above this level) reaches `target`.  All sums run in one
// fixed order, so every CTA of a cluster gets the same answer.  Results go to sh.found_bin,
// sh.mass_above, sh.mass_ge, sh.cnt_above, sh.cnt_bin.  Returns the mass of everything at
// this level plus the carry (the row total at level 1).
__device__ double scan_bins(Shared& sh, int nbins, double carry_mass, unsigned int carry_cnt,
                            double target, bool target_is_fraction, float p) {
  const int groups = nbins / kGroup;
  const int tid = threadIdx.x;
  const double* const mass = sh.mass;
  const unsigned int* const cnt = sh.cnt;
  if (tid < groups) {
    double s = 0.0;
    unsigned int c = 0;
    for (int b = kGroup - 1; b >= 0; --b) {
      s += mass[tid * kGroup + b];
      c += cnt[tid * kGroup + b];
    }
    sh.grp_mass[tid] = s;
    sh.grp_cnt[tid] = c;
  }
  __syncthreads();
  if (tid == 0) {
    double s = carry_mass;
    unsigned int c = carry_cnt;
    sh.suf_mass[groups] = s;
    sh.suf_cnt[groups] = c;
    for (int j = groups - 1; j >= 0; --j) {
      s += sh.grp_mass[j];
      c += sh.grp_cnt[j];
      sh.suf_mass[j] = s;
      sh.suf_cnt[j] = c;
    }
    sh.found_group = -1;
  }
  __syncthreads();
  const double all = sh.suf_mass[0];
  if (target_is_fraction) target = static_cast<double>(p) * all;
  if (tid < groups && sh.suf_mass[tid + 1] < target && target <= sh.suf_mass[tid])
    sh.found_group = tid;  // the suffix sums are monotone: at most one group qualifies
  __syncthreads();
  if (tid == 0) {
    int j = sh.found_group;
    if (j < 0) {  // only reachable through rounding at the very bottom: take the lowest group
      j = 0;
      while (j < groups - 1 && sh.grp_cnt[j] == 0) ++j;
    }
    double s = sh.suf_mass[j + 1];
    unsigned int c = sh.suf_cnt[j + 1];
    int found = -1;
    double prev = s;
    unsigned int cprev = c;
    int last_bin = -1;
    for (int b = kGroup - 1; b >= 0; --b) {
      const int bin = j * kGroup + b;
      const unsigned int cb = cnt[bin];
      if (cb == 0) continue;
      prev = s;
      cprev = c;
      s += mass[bin];
      c += cb;
      last_bin = bin;
      if (target <= s) {
        found = bin;
        break;
      }
    }
    if (found < 0) found = last_bin;  // rounding between the two summation orders
    if (found < 0) {                  // empty level (cannot happen with target > 0)
      found = 0;
      prev = s;
      cprev = c;
    }
    sh.found_bin = found;
    sh.mass_above = prev;
    sh.mass_ge = s;
    sh.cnt_above = cprev;
    sh.cnt_bin = c - cprev;
  }
  __syncthreads();
  return all;
}

__global__ void __launch_bounds__(kBlock, 2) select_topp_kernel(const __grid_constant__ SelectParams P) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Shared& sh = *reinterpret_cast<Shared*>(smem_raw);
  float* a = reinterpret_cast<float*>(smem_raw + ((sizeof(Shared) + 127) / 128) * 128);

  cg::cluster_group cluster = cg::this_cluster();
  const int cs = static_cast<int>(cluster.num_blocks());
  const int rank = static_cast<int>(cluster.block_rank());
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const bool worker = tid < kThreads;

  const int list = blockIdx.y;  // (used slot, sequence, group)
  const int g = list % P.G;
  const int b = (list / P.G) % P.B;
  const int slot = list / (P.G * P.B);
  const int u = P.layer_of[slot];
  const long long out_list = (static_cast<long long>(u) * P.B + b) * P.G + g;

  long long Lll = P.kv_len[b];
  if (Lll < 0) Lll = 0;
  if (Lll > P.L_stride) Lll = P.L_stride;
  const int L = static_cast<int>(Lll);
  const int per = ((L + cs - 1) / cs + 3) & ~3;  // slice length, 16-byte aligned start
  const int lo = min(L, rank * per);
  const int hi = min(L, lo + per);
  const int n_loc = hi - lo;

  // contributing rows in the order that defines the aggregated value
  if (tid == 0) {
    int n = 0;
    for (int h = 0; h < P.H; ++h) {
      if (P.has_groups && P.head_group[h] != g) continue;
      for (int s = 0; s < P.gamma; ++s) sh.row_off[n++] = static_cast<long long>(h * P.gamma + s) * P.L_stride;
    }
    sh.n_rows = n;
  }
  for (int i = tid; i < kHistSlots; i += kBlock) sh.hist[i] = 0ull;
  __syncthreads();
  const int R = sh.n_rows;

  // ---- 1+2: aggregate the slice and build the level-1 histogram ------------------------------
  const float* A = P.probs[slot] + static_cast<long long>(b) * P.H * P.gamma * P.L_stride + lo;
  const int n4 = (n_loc + 3) >> 2;
  const int n_pos4 = n4 * 4;                       // slice length rounded up to whole float4s
  const int n_chunks = (n_pos4 + kChunk - 1) / kChunk;
  // ring buffers follow the aggregated slice (whose capacity is fixed by the launch)
  const int slice_cap4 = ((((P.L_stride + cs - 1) / cs + 3) & ~3ll) + 31) & ~31ll;
  float* ring = a + slice_cap4;
  if (tid == 0) {
    sh.mass = reinterpret_cast<double*>(ring);
    sh.cnt = reinterpret_cast<unsigned int*>(ring + 2 * kL1Bins);
  }
  bool bad = false;
  // Pieces are numbered q = chunk * R + row, i.e. in the order the adds must happen.  Every
  // thread copies exactly the two float4 columns of a piece that it will add itself, with
  // 16-byte cp.async into its own ring slots, kDepth pieces ahead: completion is tracked per
  // thread (commit / wait groups), so the pipeline needs no barrier at all and holds
  // kDepth x 8 KB of reads in flight per CTA without occupying registers.
  {
    const uint32_t ring_addr = smem_u32(ring) + tid * 16;
    const float* src0 = A + 4 * tid;
    int ic = 0, ir = 0, islot = 0;  // chunk, row and ring slot of the next piece to request
    auto issue = [&]() {
      if (ic < n_chunks) {
        const int len4 = min(kChunk, n_pos4 - ic * kChunk) >> 2;
        const float* src = src0 + sh.row_off[ir] + ic * kChunk;
        const uint32_t dst = ring_addr + islot * (kChunk * 4);
#pragma unroll
        for (int k = 0; k < 2; ++k)
          if (tid + k * kThreads < len4) cp_async16(dst + k * kThreads * 16, src + k * kThreads * 4);
        if (++ir == R) { ir = 0; ++ic; }
        islot = (islot + 1) & (kDepth - 1);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    for (int q = 0; q < kDepth - 1; ++q) issue();
    // Validity of the inputs is tracked with a running minimum (a negative input, the only
    // invalid value a sum can hide) -- NaN and Inf survive into the aggregated value itself.
    float4 acc[2], mn[2];
    acc[0] = acc[1] = mn[0] = mn[1] = make_float4(0.f, 0.f, 0.f, 0.f);
    int slot = 0;
    for (int c = 0; c < n_chunks; ++c) {
      const int len4 = min(kChunk, n_pos4 - c * kChunk) >> 2;
      // positions of this thread's two float4s that lie beyond the slice (last float4 only)
      int cut[2];
#pragma unroll
      for (int k = 0; k < 2; ++k) cut[k] = n_loc - (c * kChunk + 4 * (tid + k * kThreads));
      for (int r = 0; r < R; ++r) {
        issue();
        asm volatile("cp.async.wait_group %0;" ::"n"(kDepth - 1) : "memory");
        const float4* piece = reinterpret_cast<const float4*>(ring + slot * kChunk);
        slot = (slot + 1) & (kDepth - 1);
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int i4 = tid + k * kThreads;
          if (i4 < len4) {
            float4 x = piece[i4];
            if (cut[k] < 4) {  // values beyond kv_len are not inputs
              if (cut[k] < 4) x.w = 0.f;
              if (cut[k] < 3) x.z = 0.f;
              if (cut[k] < 2) x.y = 0.f;
            }
            mn[k].x = fminf(mn[k].x, x.x);
            mn[k].y = fminf(mn[k].y, x.y);
            mn[k].z = fminf(mn[k].z, x.z);
            mn[k].w = fminf(mn[k].w, x.w);
            acc[k].x = acc[k].x + x.x;
            acc[k].y = acc[k].y + x.y;
            acc[k].z = acc[k].z + x.z;
            acc[k].w = acc[k].w + x.w;
          }
        }
      }
      // the chunk is complete: store it and feed the level-1 histogram
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int i4 = tid + k * kThreads;
        const bool act = i4 < len4;
        const int pos = c * kChunk + 4 * i4;  // position inside the slice
        const float4 v = acc[k];
        if (act) {
          *reinterpret_cast<float4*>(a + pos) = v;
          bad |= (mn[k].x < 0.f) | (mn[k].y < 0.f) | (mn[k].z < 0.f) | (mn[k].w < 0.f);
          bad |= !(v.x <= FLT_MAX) | !(v.y <= FLT_MAX) | !(v.z <= FLT_MAX) | !(v.w <= FLT_MAX);
        }
        const float vals[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned int key = __float_as_uint(vals[e]);
          // zeros carry no mass and can never be the threshold of a row with positive total
          const bool take = act && (pos + e < n_loc) && key != 0u && !(key >> 31);
          hist_add(sh.hist, take, static_cast<int>(key >> 20), mantissa_of(key));
        }
        acc[k] = mn[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  }
  if (bad) atomicAdd(&sh.hist[kInvalidSlot], 1ull);
  __syncthreads();

  // ---- 3: threshold search --------------------------------------------------------------------
  // invalid inputs anywhere in the cluster?
  cluster.sync();
  unsigned long long n_bad = 0, n_timeout = 0;
  for (int r = 0; r < cs; ++r) {
    n_bad += *cluster.map_shared_rank(&sh.hist[kInvalidSlot], r);
    n_timeout += *cluster.map_shared_rank(&sh.hist[kTimeoutSlot], r);
  }

  unsigned int theta_key = 0u;  // keep everything with key >= theta_key
  double total = 0.0, target = 0.0, m_gt = 0.0, m_ge = 0.0;
  bool invalid = (n_bad != 0) || (n_timeout != 0);
  if (!invalid) {
    // level 1: bins = top 11 bits of the (non-negative) pattern
    reduce_hist(cluster, sh, kL1Bins, [](int bin) { return max(bin >> 3, 1) - 150; });
    total = scan_bins(sh, kL1Bins, 0.0, 0u, 0.0, true, P.p);
    target = static_cast<double>(P.p) * total;
    if (target > 0.0 && !P.keep_all) {
      const int b1 = sh.found_bin;
      const int e1 = max(b1 >> 3, 1) - 150;
      unsigned int prefix = static_cast<unsigned int>(b1);
      double carry_m = sh.mass_above;
      unsigned int carry_c = sh.cnt_above;
      for (int level = 0; level < 2; ++level) {
        const int shift = (level == 0) ? 10 : 0;
        __syncthreads();
        for (int i = tid; i < kL23Bins; i += kBlock) sh.hist[i] = 0ull;
        __syncthreads();
        for (int base = 0; base < n_loc && worker; base += kThreads) {
          const int i = base + tid;
          unsigned int key = 0u;
          bool take = false;
          if (i < n_loc) {
            key = __float_as_uint(a[i]);
            take = (key >> (shift + 10)) == prefix;
          }
          hist_add(sh.hist, take, static_cast<int>((key >> shift) & 1023u), mantissa_of(key));
        }
        reduce_hist(cluster, sh, kL23Bins, [e1](int) { return e1; });
        scan_bins(sh, kL23Bins, carry_m, carry_c, target, false, P.p);
        prefix = (prefix << 10) | static_cast<unsigned int>(sh.found_bin);
        carry_m = sh.mass_above;
        carry_c = sh.cnt_above;
      }
      theta_key = prefix;
      m_gt = sh.mass_above;
      m_ge = sh.mass_ge;
    } else {
      m_ge = total;  // p >= 1, or an all-zero row where everything ties at zero: keep all
    }
  }

  // ---- 4: ordered compaction --------------------------------------------------------------------
  // per-warp contiguous chunks of the slice, 32 positions per step
  const int chunk = (((n_loc + kWarps - 1) / kWarps) + 31) & ~31;
  const int w_lo = min(n_loc, warp * chunk);
  const int w_hi = min(n_loc, w_lo + chunk);
  int wc = 0;
  if (!invalid && worker) {
    for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
      const int i = i0 + lane;
      const bool keep = i < w_hi && __float_as_uint(a[i]) >= theta_key;
      wc += __popc(__ballot_sync(0xffffffffu, keep));
    }
  }
  if (lane == 0 && worker) sh.warp_cnt[warp] = wc;
  __syncthreads();
  if (tid == 0) {
    int s = 0;
    for (int w = 0; w < kWarps; ++w) {
      const int c = sh.warp_cnt[w];
      sh.warp_cnt[w] = s;
      s += c;
    }
    sh.local_kept = s;
  }
  cluster.sync();  // local_kept of every CTA is visible
  long long offset = 0, count = 0;
  for (int r = 0; r < cs; ++r) {
    const int c = *cluster.map_shared_rank(&sh.local_kept, r);
    if (r < rank) offset += c;
    count += c;
  }
  if (!invalid && worker) {
    int* out = P.idx + out_list * P.idx_stride;
    long long pos = offset + sh.warp_cnt[warp];
    for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
      const int i = i0 + lane;
      const bool keep = i < w_hi && __float_as_uint(a[i]) >= theta_key;
      const unsigned m = __ballot_sync(0xffffffffu, keep);
      const long long my = pos + __popc(m & ((1u << lane) - 1u));
      if (keep && my < P.idx_stride) out[my] = lo + i;
      pos += __popc(m);
    }
  }
  if (rank == 0 && tid == 0) {
    int st = SPECATTN_ROW_OK;
    if (invalid) {
      st = (n_bad != 0 ? SPECATTN_ROW_INVALID_PROB : 0) | (n_timeout != 0 ? SPECATTN_ROW_TIMEOUT : 0);
      count = 0;
    } else if (count > P.idx_stride) {
      st = SPECATTN_ROW_OVERFLOW;
    }
    P.counts[out_list] = static_cast<int>(count);
    P.status[out_list] = st;
    if (P.diag != nullptr) {
      double* d = P.diag + out_list * 4;
      d[0] = total;
      d[1] = target;
      d[2] = m_gt;
      d[3] = m_ge;
    }
  }
  cluster.sync();  // nobody leaves while its shared memory may still be read remotely
}

int pick_cluster(long long L_stride, long long n_lists) {
  int cs = 1;
  while (cs < 8 && (L_stride + cs - 1) / cs > 8192) cs *= 2;
  while (cs < 8 && n_lists * cs < 296 && L_stride / cs > 512) cs *= 2;
  return cs;
}

}  // namespace
}  // namespace specattn

using specattn::SelectParams;

extern "C" int specattn_select_topp(const specattn_select_args* args, void* cuda_stream) {
  if (args == nullptr) return SPECATTN_ERR_NULL;
  if (args->struct_size != sizeof(specattn_select_args)) return SPECATTN_ERR_STRUCT_SIZE;
  const specattn_select_args& A = *args;
  if (!A.draft_probs || !A.kv_len || !A.layer_map || !A.idx || !A.counts || !A.row_status)
    return SPECATTN_ERR_NULL;
  if (A.n_draft_layers < 1 || A.n_draft_layers > SPECATTN_MAX_DRAFT_LAYERS) return SPECATTN_ERR_RANGE;
  if (A.n_target_layers < 0 || A.batch < 0 || A.gamma < 1 || A.n_groups < 1) return SPECATTN_ERR_RANGE;
  if (A.n_draft_heads < 1 || A.n_draft_heads > SPECATTN_MAX_DRAFT_HEADS) return SPECATTN_ERR_RANGE;
  if (A.L_stride < 0 || A.idx_stride < 0) return SPECATTN_ERR_RANGE;
  if (!(A.p > 0.0f)) return SPECATTN_ERR_RANGE;  // also rejects NaN
  if (A.L_stride % 4 != 0) return SPECATTN_ERR_ALIGN;
  if (A.L_stride > SPECATTN_MAX_KV_LEN) return SPECATTN_ERR_UNSUPPORTED;
  if (static_cast<long long>(A.n_draft_heads) * A.gamma > SPECATTN_MAX_ROWS_PER_LIST)
    return SPECATTN_ERR_UNSUPPORTED;

  SelectParams P;
  memset(&P, 0, sizeof(P));
  bool used[SPECATTN_MAX_DRAFT_LAYERS] = {false};
  for (int j = 0; j < A.n_target_layers; ++j) {
    const int u = A.layer_map[j];
    if (u < -1 || u >= A.n_draft_layers) return SPECATTN_ERR_RANGE;
    if (u >= 0) used[u] = true;
  }
  int n_used = 0;
  for (int u = 0; u < A.n_draft_layers; ++u) {
    if (!used[u]) continue;
    if (A.draft_probs[u] == nullptr) return SPECATTN_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(A.draft_probs[u]) % 16 != 0) return SPECATTN_ERR_ALIGN;
    P.probs[n_used] = A.draft_probs[u];
    P.layer_of[n_used] = u;
    ++n_used;
  }
  if (A.head_group != nullptr) {
    for (int h = 0; h < A.n_draft_heads; ++h) {
      if (A.head_group[h] < 0 || A.head_group[h] >= A.n_groups) return SPECATTN_ERR_RANGE;
      P.head_group[h] = static_cast<signed char>(A.head_group[h] & 0x7f);
      if (A.head_group[h] > 127) return SPECATTN_ERR_UNSUPPORTED;
    }
    P.has_groups = 1;
  }
  const long long n_lists = static_cast<long long>(n_used) * A.batch * A.n_groups;
  if (n_lists == 0) return SPECATTN_OK;
  if (n_lists > 65535) return SPECATTN_ERR_UNSUPPORTED;

  P.n_used = n_used;
  P.B = A.batch;
  P.H = A.n_draft_heads;
  P.gamma = A.gamma;
  P.G = A.n_groups;
  P.L_stride = A.L_stride;
  P.kv_len = A.kv_len;
  P.p = A.p;
  P.keep_all = (A.p >= 1.0f) ? 1 : 0;
  P.idx = A.idx;
  P.idx_stride = A.idx_stride;
  P.counts = A.counts;
  P.status = A.row_status;
  P.diag = A.diag;

  const int cs = specattn::pick_cluster(A.L_stride, n_lists);
  const long long slice = (((A.L_stride + cs - 1) / cs) + 3) / 4 * 4;
  if (slice > specattn::kSliceCap) return SPECATTN_ERR_UNSUPPORTED;
  // shared memory: fixed part, the aggregated slice, then the per-thread staging ring
  // (kDepth pieces of 8 KB; it later hosts the reduced histogram).  Small slices leave room
  // for two CTAs per SM.
  const size_t fixed = ((sizeof(specattn::Shared) + 127) / 128) * 128;
  const size_t slice_bytes = static_cast<size_t>((slice + 31) / 32 * 32) * sizeof(float);
  const size_t smem = fixed + slice_bytes + static_cast<size_t>(specattn::kDepth) * specattn::kChunk * sizeof(float);
  if (smem > 224 * 1024) return SPECATTN_ERR_UNSUPPORTED;

  // Opt in to large dynamic shared memory once per device, so that later calls issue nothing
  // but the launch.
  cudaError_t err = cudaSuccess;
  {
    static std::atomic<unsigned long long> done_mask{0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPECATTN_ERR_CUDA;
    if (!((done_mask.load(std::memory_order_acquire) >> dev) & 1ull)) {
      err = cudaFuncSetAttribute(specattn::select_topp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 224 * 1024);
      if (err != cudaSuccess) {
        cudaGetLastError();
        return SPECATTN_ERR_CUDA;
      }
      done_mask.fetch_or(1ull << dev, std::memory_order_release);
    }
  }

  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(static_cast<unsigned>(cs), static_cast<unsigned>(n_lists), 1);
  cfg.blockDim = dim3(specattn::kBlock, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = static_cast<cudaStream_t>(cuda_stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(cs);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  err = cudaLaunchKernelEx(&cfg, specattn::select_topp_kernel, P);
  if (err != cudaSuccess) {
    cudaGetLastError();
    return SPECATTN_ERR_CUDA;
  }
  specattn::g_launch_count.fetch_add(1, std::memory_order_relaxed);
  return SPECATTN_OK;
}
