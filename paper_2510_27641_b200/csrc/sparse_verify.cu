// specattn_sparse_verify: grouped-query sparse decode attention of the gamma+1 verification
// queries over the selected rows of a paged bf16 K/V cache, for sm_100a.
//
// Paper: Eq. 1 restricted to the index set I of Eq. 2-3 (normalised over I), Sec. 3.5, and
// Alg. 1's "Verification with Sparse Attention" (one list per layer, shared by all gamma+1
// queries and by all heads of a GQA group).  The paper feeds a CSR mask to a library
// block-sparse kernel; here the ascending index lists are consumed directly.
//
// Mapping to the GPU.  The work of a call is the list of (sequence, kv head) units, unit u
// holding count(u) tokens; it is cut into atoms of 16 tokens and the atoms are dealt evenly
// and contiguously to one persistent CTA per SM, so ragged batches balance without any host
// knowledge of the counts.  Inside a CTA
//   - four producer warps resolve position -> (page, slot) through the block table and fetch
//     each selected 256-byte K row and V row with 16-byte cp.async copies (16 lanes per row,
//     completion counted on an mbarrier) into a padded, bank-conflict-free shared-memory tile;
//     a 4-stage ring of 64-token tiles guarded by full/empty mbarriers keeps >100 KB of reads
//     in flight per SM.  (One 1-D bulk copy per row was measured first: the TMA unit retires
//     about one such 256-byte request per 19 cycles per SM, capping the gather near 3.4 TB/s.)
//   - the consumer warps own one 16-row slab of the (gamma+1) x group query block; the warps of
//     a slab take alternate tiles (and, four to a slab, one 32-key half of them), so each warp
//     runs long independent chains: S = Q K^T and O += P V on the tensor cores (bf16 mma.sync,
//     fp32 accumulate; P is split into two bf16 terms so that it carries 16 mantissa bits),
//     online softmax in fp32 registers in the log2 domain;
//   - at the end of a unit the warps of a slab combine through shared memory; a unit that was
//     cut between CTAs is finished by whichever CTA arrives last at the unit's counter, which
//     merges all partial (O, m, l) records in a fixed order -- nobody ever waits on a peer.
// Every mbarrier wait is bounded; on expiry the CTA flags SPECATTN_ROW_TIMEOUT and leaves.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <atomic>

#include "ptx.cuh"
#include "nvtx_range.h"
#include "specattn.h"

namespace specattn {

extern std::atomic<long long> g_launch_count;
int device_sm_count();

namespace {

constexpr int kD = 128;            // head dimension
constexpr int kRowBytes = kD * 2;  // one K or V row of one head
constexpr int kPitch = kRowBytes + 16;  // shared-memory row pitch: ldmatrix hits 8 distinct 16-byte lanes
constexpr int kStageTok = 64;
constexpr int kStages = 4;
constexpr int kProdWarps = 4;  // one per stage
constexpr int kAtom = 16;
constexpr int kMaxUnits = SPECATTN_MAX_VERIFY_UNITS;
constexpr int kRec = 68 * 32;  // floats of one warp's (acc[64], m0, l0, m1, l1) record, lane-major
constexpr int kCountersPerUnit = 4;
constexpr int kAlignedMaxUnits = 256;  // the unit-aligned partition is tried up to this many units
constexpr int kCandidates = 8;         // candidate target shares tried for it
// A unit is not cut into parts of fewer than this many atoms (two 64-token tiles) even when
// there are CTAs to spare: every part costs a record, an arrival and a share of the merge, which
// on a small call (one short sequence) outweighs the streaming time saved.
constexpr int kMinPartAtoms = 8;
// With CTA pairs available (query blocks of up to 32 rows), a unit of up to this many atoms is cut
// in two rather than in more parts: the pair's merge through shared memory (~1.7 us) beats the
// merge of three or more records through global memory (~1 us per record) by more than the
// longer parts cost.
constexpr int kPairAtoms = 64;
constexpr size_t kCounterBytes = static_cast<size_t>(kMaxUnits) * kCountersPerUnit * sizeof(unsigned int);
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kLog2e = 1.4426950408889634f;

struct VerifyParams {
  int B, T, Hq, Hkv, grp, M, G, dense;
  int page_size, page_shift;  // page_shift >= 0 when page_size is a power of two
  const __nv_bfloat16* q;
  const __nv_bfloat16* kv;
  long long n_pages, s_page, s_kv, s_slot, s_head;
  const int* bt;
  long long bt_stride;
  const int* kv_len;
  const int* idx;
  long long idx_stride;
  const int* counts;
  float scale_log2;
  float* out;
  float* lse;
  int* status;
  unsigned int* counters;
  float* partials;
  int lists_stable;  // SPECATTN_VERIFY_LISTS_STABLE
  int tail;          // in-flight tokens appended to every unit, attended causally
  int tail_off;      // tail - T: query t may see tail tokens j <= t + tail_off
  const int* plan;   // precomputed work partition (specattn_verify_plan) or nullptr
  int test_lose;     // SPECATTN_VERIFY_TEST_LOSE_ARRIVAL: CTA 0 withholds one barrier arrival
  int pairs;         // the launch runs as CTA pairs (clusters of two)
};

// WPM = consumer warps per 16-row slab: 4 -> (stage parity, 32-key half), 2 -> (stage parity).
template <int MT, int WPM>
struct VShared {
  alignas(128) unsigned char kv[kStages][2][kStageTok * kPitch];
  alignas(16) unsigned char q[MT * 16 * kPitch];
  alignas(16) float scratch[MT][WPM / 2][kRec];
  alignas(8) unsigned long long full[kStages];
  unsigned long long empty[kStages];
  unsigned long long q_full, q_empty;
  int unit_start[kMaxUnits + 1];
  int unit_cnt[kMaxUnits];
  int part_start[kAlignedMaxUnits + 1];  // aligned partition: first CTA of each unit
  int cand_parts[kCandidates];           // per candidate share: total parts, largest part
  int cand_max[kCandidates];
  int aligned;                           // 1: unit-aligned partition, 0: contiguous atoms
  volatile int abort_flag;
  // (kernels with two warps per slab) this CTA arrived last at the cut unit of its final segment:
  // both warps of the slab merge half of the columns each; with the merge's arguments
  volatile int merge_last[MT];
  volatile int merge_arg[MT][5];
  // cluster merge (two CTAs per unit): the odd CTA's records land here, in the even CTA
  unsigned long long peer_full;
  alignas(16) float peer_rec[(MT <= 2) ? MT : 1][(MT <= 2) ? kRec : 1];
};

__device__ __forceinline__ int unit_count(const VerifyParams& P, int u) {
  const int b = u / P.Hkv;
  long long c;
  if (P.dense) {
    c = P.kv_len[b];
  } else {
    const int g = (P.G == 1) ? 0 : (u % P.Hkv);
    c = P.counts[static_cast<long long>(b) * P.G + g];
    if (c > P.idx_stride) c = P.idx_stride;
  }
  if (c < 0) c = 0;
  return static_cast<int>(c) + P.tail;  // the in-flight tokens follow the list
}

// First atom of CTA i when n atoms are dealt to np CTAs.
__device__ __forceinline__ int cta_first_atom(long long i, long long n, long long np) {
  return static_cast<int>(i * n / np);
}
// The CTA that owns atom x.
__device__ __forceinline__ int cta_of_atom(long long x, long long n, long long np) {
  long long i = ((x + 1) * np + n - 1) / n - 1;
  if (i > np - 1) i = np - 1;
  return static_cast<int>(i);
}

// Scales that bring a running maximum m and an incoming maximum im to their common maximum.
__device__ __forceinline__ void merge_scales(float m, float im, float& mn, float& a_old, float& a_in) {
  mn = fmaxf(m, im);
  const float base = (mn == -INFINITY) ? 0.f : mn;
  a_old = ex2(m - base);   // ex2(-inf) = 0
  a_in = ex2(im - base);
}

// ---- precomputed work partition ("plan") ------------------------------------------------------
// The partition of a launch depends only on the list lengths, the shapes and the grid: target
// layers that share a draft layer's lists share it.  A plan holds, as int32:
//   [0] magic  [1] U  [2] grid  [3] aligned  [4] NP  [5] N (atoms)  [6] tail  [7] dense
//   unit_start[U + 1], unit_cnt[U], part_start[U + 1], then (a0, a1, u_first) per CTA
// A kernel whose launch does not match the header ignores the plan and partitions itself.
constexpr int kPlanMagic = 0x5a17a9e1;
constexpr int kPlanHeader = 8;
__host__ __device__ inline size_t plan_ints(int U, int grid) {
  return static_cast<size_t>(kPlanHeader) + (U + 1) + U + (U + 1) + 3 * static_cast<size_t>(grid);
}

// One CTA computes what every CTA of a verify launch would compute for itself at start-up.
__device__ __forceinline__ void plan_body(const VerifyParams& P, int* plan, int G) {
  __shared__ int unit_start[kMaxUnits + 1];
  __shared__ int part_start[kAlignedMaxUnits + 1];
  __shared__ int cand_parts[kCandidates], cand_max[kCandidates];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int U = P.B * P.Hkv;
  // The lists are the previous kernel's output.  No early trigger for the next kernel either:
  // a verify launch flagged SPECATTN_VERIFY_LISTS_STABLE reads the plan without waiting, so it
  // must not be scheduled before this grid has completed (completion is the trigger).
  pdl_wait();
  int* const p_us = plan + kPlanHeader;
  int* const p_cnt = p_us + (U + 1);
  int* const p_ps = p_cnt + U;
  int* const p_cta = p_ps + (U + 1);
  if (tid == 0) unit_start[0] = 0;
  for (int u = tid; u < U; u += 256) {
    const int c = unit_count(P, u);
    p_cnt[u] = c;
    unit_start[u + 1] = (c + kAtom - 1) / kAtom;
  }
  if (tid < kCandidates) { cand_parts[tid] = 0; cand_max[tid] = 0; }
  __syncthreads();
  if (warp == 0) {
    int carry = 0;
    for (int base = 0; base < U; base += 32) {
      const int u = base + lane;
      int v = (u < U) ? unit_start[u + 1] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += n;
      }
      if (u < U) unit_start[u + 1] = v + carry;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  }
  __syncthreads();
  const long long N = unit_start[U];
  const bool try_aligned = (U <= kAlignedMaxUnits) && (N > 0);
  if (try_aligned && tid < U) {
    const int atoms = unit_start[tid + 1] - unit_start[tid];
    if (atoms > 0) {
      for (int c = 0; c < kCandidates; ++c) {
        const unsigned int num = static_cast<unsigned int>(atoms) * G * 16u;
        const unsigned int den = static_cast<unsigned int>(N) * (16u + c);
        int k = static_cast<int>((2u * num + den) / (2u * den));
        if (k < 1) k = 1;
        if (k > atoms) k = atoms;
        if (k * kMinPartAtoms > atoms) k = max(1, atoms / kMinPartAtoms);  // no part shorter than that
        if (P.pairs && k > 2 && atoms <= kPairAtoms) k = 2;  // short unit: two parts merge through shared memory
        atomicAdd(&cand_parts[c], k);
        atomicMax(&cand_max[c], (atoms + k - 1) / k);
      }
    }
  }
  __syncthreads();
  int cand = -1;
  if (try_aligned) {
    for (int c = 0; c < kCandidates; ++c)
      if (cand_parts[c] <= G) { cand = c; break; }
    if (cand >= 0 && static_cast<long long>(cand_max[cand]) * G > N + 24ll * G) cand = -1;
  }
  const bool aligned = cand >= 0;
  if (aligned && warp == 0) {
    int carry = 0;
    for (int base = 0; base < U; base += 32) {
      const int u = base + lane;
      int k = 0;
      if (u < U) {
        const int atoms = unit_start[u + 1] - unit_start[u];
        if (atoms > 0) {
          const unsigned int num = static_cast<unsigned int>(atoms) * G * 16u;
          const unsigned int den = static_cast<unsigned int>(N) * (16u + cand);
          k = static_cast<int>((2u * num + den) / (2u * den));
          if (k < 1) k = 1;
          if (k > atoms) k = atoms;
        if (k * kMinPartAtoms > atoms) k = max(1, atoms / kMinPartAtoms);  // no part shorter than that
        if (P.pairs && k > 2 && atoms <= kPairAtoms) k = 2;  // short unit: two parts merge through shared memory
        }
      }
      int v = k;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += n;
      }
      if (u < U) part_start[u + 1] = v + carry;
      if (base == 0 && lane == 0) part_start[0] = 0;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  }
  __syncthreads();
  const long long NP = aligned ? part_start[U] : ((N < G) ? N : static_cast<long long>(G));
  for (int u = tid; u <= U; u += 256) {
    p_us[u] = unit_start[u];
    p_ps[u] = aligned ? part_start[u] : 0;
  }
  for (int i = tid; i < G; i += 256) {
    int a0 = 0, a1 = 0, u_first = 0;
    if (i < NP) {
      if (aligned) {
        int lo = 0, hi = U - 1;
        while (lo < hi) {
          const int mid = (lo + hi + 1) >> 1;
          if (part_start[mid] <= i) lo = mid; else hi = mid - 1;
        }
        const int k = part_start[lo + 1] - part_start[lo];
        const int j = i - part_start[lo];
        const int atoms = unit_start[lo + 1] - unit_start[lo];
        a0 = unit_start[lo] + j * atoms / k;
        a1 = unit_start[lo] + (j + 1) * atoms / k;
      } else {
        a0 = cta_first_atom(i, N, NP);
        a1 = cta_first_atom(i + 1, N, NP);
      }
      int lo = 0, hi = U - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (unit_start[mid] <= a0) lo = mid; else hi = mid - 1;
      }
      u_first = lo;
      while (unit_start[u_first + 1] <= a0) ++u_first;
    }
    p_cta[3 * i] = a0;
    p_cta[3 * i + 1] = a1;
    p_cta[3 * i + 2] = u_first;
  }
  if (tid == 0) {
    plan[1] = U;
    plan[2] = G;
    plan[3] = aligned ? 1 : 0;
    plan[4] = static_cast<int>(NP);
    plan[5] = static_cast<int>(N);
    plan[6] = P.tail;
    plan[7] = P.dense;
    plan[0] = kPlanMagic;
  }
}

__global__ void __launch_bounds__(256, 1) verify_plan_kernel(const __grid_constant__ VerifyParams P, int* plan, int G) {
  plan_body(P, plan, G);
}

// The plans of several launches (one per draft layer whose lists the step's layers share) in
// one launch, one CTA each.
constexpr int kPlanBatch = 8;
struct PlanBatch {
  VerifyParams p[kPlanBatch];
  int* plan[kPlanBatch];
  int G;
};
__global__ void __launch_bounds__(256, 1) verify_plan_many_kernel(const __grid_constant__ PlanBatch B) {
  plan_body(B.p[blockIdx.x], B.plan[blockIdx.x], B.G);
}

// Online-softmax state of one warp: rows g and g+8 of its 16-row slab, 128 output columns.
struct WarpState {
  float acc[16][4];
  float m0, m1, l0, l1;
};

// One 32-key block: S = Q K^T (4 n-tiles), online softmax, O += P V with P = P_hi + P_lo.
// `valid` = number of existing keys in the block (>= 1; rows beyond it hold finite padding).
// `tail_begin` = index inside the block of the first in-flight token (>= 32: none); rows g and
// g+8 of the slab may see in-flight tokens j <= lim0 / lim1 only (causal among themselves).
template <bool kQReload>
__device__ __forceinline__ void attend_block32(WarpState& st, const uint32_t (&qf)[8][4], uint32_t q_addr, uint32_t k_addr,
                                               uint32_t v_addr, int valid, float scale_log2, int tq,
                                               int tail_begin, int lim0, int lim1) {
  float sc[4][4];
#pragma unroll
  for (int n = 0; n < 4; ++n) sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f;
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    uint32_t qa[4], k0[4], k1[4];
    if (kQReload) {
      ldmatrix_x4(qa, q_addr + kk * 32);
    } else {
      qa[0] = qf[kk][0];
      qa[1] = qf[kk][1];
      qa[2] = qf[kk][2];
      qa[3] = qf[kk][3];
    }
    ldmatrix_x4(k0, k_addr + kk * 32);
    ldmatrix_x4(k1, k_addr + 16 * kPitch + kk * 32);
    mma_bf16(sc[0], qa, k0[0], k0[1]);
    mma_bf16(sc[1], qa, k0[2], k0[3]);
    mma_bf16(sc[2], qa, k1[0], k1[1]);
    mma_bf16(sc[3], qa, k1[2], k1[3]);
  }
  // raw scores stay unscaled: exp2(s * c - m * c) is one fused multiply-add per element
  if (valid < 32) {  // only the last block of a segment has missing keys
#pragma unroll
    for (int n = 0; n < 4; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int key = n * 8 + tq * 2 + (i & 1);
        if (key >= valid) sc[n][i] = -INFINITY;
      }
  }
  if (tail_begin < 32) {  // the block holds in-flight tokens: causal mask per query row
#pragma unroll
    for (int n = 0; n < 4; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int j = n * 8 + tq * 2 + (i & 1) - tail_begin;
        if (j >= 0 && j > ((i & 2) ? lim1 : lim0)) sc[n][i] = -INFINITY;  // j < 0: a listed row
      }
  }
  float mx0 = fmaxf(fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1])),
                    fmaxf(fmaxf(sc[2][0], sc[2][1]), fmaxf(sc[3][0], sc[3][1])));
  float mx1 = fmaxf(fmaxf(fmaxf(sc[0][2], sc[0][3]), fmaxf(sc[1][2], sc[1][3])),
                    fmaxf(fmaxf(sc[2][2], sc[2][3]), fmaxf(sc[3][2], sc[3][3])));
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
  // running maxima are kept in the scaled log2 domain (scale_log2 > 0 keeps the order)
  const float mn0 = fmaxf(st.m0, mx0 * scale_log2), mn1 = fmaxf(st.m1, mx1 * scale_log2);
  const float base0 = (mn0 == -INFINITY) ? 0.f : mn0;
  const float base1 = (mn1 == -INFINITY) ? 0.f : mn1;
  const float al0 = ex2(st.m0 - base0), al1 = ex2(st.m1 - base1);
  st.m0 = mn0;
  st.m1 = mn1;
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int n = 0; n < 4; ++n) {
    sc[n][0] = ex2(fmaf(sc[n][0], scale_log2, -base0));
    sc[n][1] = ex2(fmaf(sc[n][1], scale_log2, -base0));
    sc[n][2] = ex2(fmaf(sc[n][2], scale_log2, -base1));
    sc[n][3] = ex2(fmaf(sc[n][3], scale_log2, -base1));
    s0 += sc[n][0] + sc[n][1];
    s1 += sc[n][2] + sc[n][3];
  }
  st.l0 = st.l0 * al0 + s0;
  st.l1 = st.l1 * al1 + s1;
  if (__any_sync(0xffffffffu, al0 != 1.f || al1 != 1.f)) {
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      st.acc[n][0] *= al0;
      st.acc[n][1] *= al0;
      st.acc[n][2] *= al1;
      st.acc[n][3] *= al1;
    }
  }
  // A-operand fragments of P for the two 16-key halves, each as a bf16 pair (hi, lo):
  // hi = bf16x2(x, y); the residuals x - hi.x, y - hi.y are exact in fp32 and rounded once more
  uint32_t phi[2][4], plo[2][4];
#pragma unroll
  for (int kb = 0; kb < 2; ++kb)
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int hrow = 0; hrow < 2; ++hrow) {
        const float x = sc[kb * 2 + n][hrow * 2], y = sc[kb * 2 + n][hrow * 2 + 1];
        const uint32_t h = pack_bf16(x, y);
        phi[kb][n * 2 + hrow] = h;
        plo[kb][n * 2 + hrow] = pack_bf16(x - __uint_as_float(h << 16), y - __uint_as_float(h & 0xffff0000u));
      }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    uint32_t v0[4], v1[4];
    ldmatrix_x4_trans(v0, v_addr + j * 32);
    ldmatrix_x4_trans(v1, v_addr + 16 * kPitch + j * 32);
    mma_bf16(st.acc[2 * j], phi[0], v0[0], v0[1]);
    mma_bf16(st.acc[2 * j + 1], phi[0], v0[2], v0[3]);
    mma_bf16(st.acc[2 * j], phi[1], v1[0], v1[1]);
    mma_bf16(st.acc[2 * j + 1], phi[1], v1[2], v1[3]);
    mma_bf16(st.acc[2 * j], plo[0], v0[0], v0[1]);
    mma_bf16(st.acc[2 * j + 1], plo[0], v0[2], v0[3]);
    mma_bf16(st.acc[2 * j], plo[1], v1[0], v1[1]);
    mma_bf16(st.acc[2 * j + 1], plo[1], v1[2], v1[3]);
  }
}

// Merge of a unit cut across CTAs by the CTA that arrived last, for one half of the 128 output
// columns (8 blocks of 8) and one warp: the common maxima of all records (four per round trip),
// then one scaled accumulation pass in CTA order with two records' half rows in flight, then rows
// g and g + 8 of slab mt written out (half 0 also writes the LSE).  Used by the kernels with two
// warps per slab, whose second warp has nothing left to do on a CTA's last segment; kept out of
// line so that it costs the tile loop no registers.
template <int MT>
__device__ __noinline__ void merge_half(const VerifyParams& P, int mt, int half, int i_lo, int i_hi, bool aligned,
                                        long long N, long long NP, int us, int b, int kvh) {
  const int lane = threadIdx.x & 31, g = lane >> 2, tq = lane & 3;
  auto record = [&](int i) -> const float4* {
    return reinterpret_cast<const float4*>(P.partials +
        (static_cast<size_t>(2 * i + ((aligned || cta_first_atom(i, N, NP) >= us) ? 0 : 1)) * MT + mt) * kRec) + lane;
  };
  float m0 = -INFINITY, m1 = -INFINITY;
  for (int i = i_lo; i <= i_hi; i += 4) {
    float4 ml[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) ml[j] = __ldcg(record(min(i + j, i_hi)) + 16 * 32);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      m0 = fmaxf(m0, ml[j].x);
      m1 = fmaxf(m1, ml[j].z);
    }
  }
  const float base0 = (m0 == -INFINITY) ? 0.f : m0, base1 = (m1 == -INFINITY) ? 0.f : m1;
  float l0 = 0.f, l1 = 0.f;
  float o[8][4];
#pragma unroll
  for (int n = 0; n < 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
  for (int i = i_lo; i <= i_hi; i += 2) {
    const bool two = i + 1 <= i_hi;
    const float4* ra = record(i);
    const float4* rb = record(two ? i + 1 : i);
    const float4 mla = __ldcg(ra + 16 * 32), mlb = __ldcg(rb + 16 * 32);
    float4 xa[8], xb[8];
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      xa[n] = __ldcg(ra + (half * 8 + n) * 32);
      xb[n] = __ldcg(rb + (half * 8 + n) * 32);
    }
    const float wa0 = ex2(mla.x - base0), wa1 = ex2(mla.z - base1);
    const float wb0 = two ? ex2(mlb.x - base0) : 0.f, wb1 = two ? ex2(mlb.z - base1) : 0.f;
    l0 += mla.y * wa0;
    l1 += mla.w * wa1;
    if (two) {
      l0 += mlb.y * wb0;
      l1 += mlb.w * wb1;
    }
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      o[n][0] += xa[n].x * wa0;
      o[n][1] += xa[n].y * wa0;
      o[n][2] += xa[n].z * wa1;
      o[n][3] += xa[n].w * wa1;
      if (two) {
        o[n][0] += xb[n].x * wb0;
        o[n][1] += xb[n].y * wb0;
        o[n][2] += xb[n].z * wb1;
        o[n][3] += xb[n].w * wb1;
      }
    }
  }
  const float inv0 = (l0 > 0.f) ? 1.f / l0 : 0.f;
  const float inv1 = (l1 > 0.f) ? 1.f / l1 : 0.f;
  const int r0 = mt * 16 + g, r1 = r0 + 8;
  if (r0 < P.M) {
    const int t = r0 / P.grp, h = kvh * P.grp + r0 % P.grp;
    const long long row = (static_cast<long long>(b) * P.T + t) * P.Hq + h;
    float* op = P.out + row * kD + tq * 2;
#pragma unroll
    for (int n = 0; n < 8; ++n)
      *reinterpret_cast<float2*>(op + (half * 8 + n) * 8) = make_float2(o[n][0] * inv0, o[n][1] * inv0);
    if (half == 0 && tq == 0) P.lse[row] = (l0 > 0.f) ? (m0 + log2f(l0)) * kLn2 : -INFINITY;
  }
  if (r1 < P.M) {
    const int t = r1 / P.grp, h = kvh * P.grp + r1 % P.grp;
    const long long row = (static_cast<long long>(b) * P.T + t) * P.Hq + h;
    float* op = P.out + row * kD + tq * 2;
#pragma unroll
    for (int n = 0; n < 8; ++n)
      *reinterpret_cast<float2*>(op + (half * 8 + n) * 8) = make_float2(o[n][2] * inv1, o[n][3] * inv1);
    if (half == 0 && tq == 0) P.lse[row] = (l1 > 0.f) ? (m1 + log2f(l1)) * kLn2 : -INFINITY;
  }
}

template <int MT, int WPM>
__global__ void __launch_bounds__((MT * WPM + kProdWarps) * 32, 1)
sparse_verify_kernel(const __grid_constant__ VerifyParams P) {
  using Sh = VShared<MT, WPM>;
  constexpr int NC = MT * WPM;                 // consumer warps
  constexpr int NT = (NC + kProdWarps) * 32;   // threads
  constexpr int NCS = MT * (WPM / 2);          // consumer warps that read any one stage
  extern __shared__ __align__(128) unsigned char smem_raw[];
  Sh& sh = *reinterpret_cast<Sh*>(smem_raw);

  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const int U = P.B * P.Hkv;
  constexpr bool kQReload = (WPM == 2);   // query fragments re-read from shared memory per block
  constexpr bool kDirectQ = true;         // consumers fetch the CTA's first query block themselves

  // Unless the caller vouched for the lists, nothing is read before the previous kernel is
  // done.  Only then may the next kernel of the stream be scheduled: a successor that starts
  // early therefore never overtakes the producer of the lists.
  if (!P.lists_stable) pdl_wait();
  pdl_launch_dependents();

  // ---- set-up: barriers, zero padding rows of the query tile, unit prefix ---------------------
  {
    uint4* zq = reinterpret_cast<uint4*>(sh.q);
    for (int i = tid; i < static_cast<int>(sizeof(sh.q) / 16); i += NT) zq[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sh.full[s], 32);   // one deferred arrival per producer lane
      mbar_init(&sh.empty[s], NCS);
    }
    mbar_init(&sh.q_full, 1);
    mbar_init(&sh.q_empty, NC);
    mbar_init(&sh.peer_full, MT);
    mbar_fence_init();
    sh.abort_flag = 0;
    sh.unit_start[0] = 0;
  }
  // A plan made for this launch (same units, grid, tail, dense flag) replaces the whole
  // partition below by one coalesced copy.
  const int* const plan = P.plan;
  const bool planned = plan != nullptr && plan[0] == kPlanMagic && plan[1] == U &&
                       plan[2] == static_cast<int>(gridDim.x) && plan[6] == P.tail && plan[7] == P.dense;
  if (planned) {
    const int* const p_us = plan + kPlanHeader;
    const int* const p_cnt = p_us + (U + 1);
    const int* const p_ps = p_cnt + U;
    for (int u = tid; u <= U; u += NT) {
      sh.unit_start[u] = p_us[u];
      if (u < U) sh.unit_cnt[u] = p_cnt[u];
      if (u <= kAlignedMaxUnits) sh.part_start[u] = p_ps[u];
    }
  } else {
    for (int u = tid; u < U; u += NT) {
      const int c = unit_count(P, u);
      sh.unit_cnt[u] = c;
      sh.unit_start[u + 1] = (c + kAtom - 1) / kAtom;
    }
  }
  fence_proxy_async();
  __syncthreads();
  // Launched as CTA pairs: the peer's barrier must exist before anyone can arrive on it.  Only
  // the arrival happens here; every thread waits for the peer's arrival where it first needs
  // it (the consumers before their first combine, everybody else before leaving), so that the
  // barrier costs nothing on the way to the first copy.
  const bool paired = (MT <= 2) && (cluster_num_ctas() == 2);
  if (paired) cluster_arrive();
  long long N;        // atoms of all units
  bool aligned;       // which of the two partitions
  long long NP;       // CTAs that get work
  int a0 = 0, a1 = 0, u_first = 0;  // this CTA's atom range and the unit holding its first atom
  const int G = static_cast<int>(gridDim.x);
  if (planned) {
    N = plan[5];
    aligned = plan[3] != 0;
    NP = plan[4];
    const int* const p_cta = plan + kPlanHeader + (U + 1) + U + (U + 1) + 3 * blockIdx.x;
    a0 = p_cta[0];
    a1 = p_cta[1];
    u_first = p_cta[2];
  } else {
  if (warp == 0) {  // inclusive scan of the atom counts, 32 at a time
    int carry = 0;
    for (int base = 0; base < U; base += 32) {
      const int u = base + lane;
      int v = (u < U) ? sh.unit_start[u + 1] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += n;
      }
      if (u < U) sh.unit_start[u + 1] = v + carry;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  }
  __syncthreads();

  // ---- work partition ----------------------------------------------------------------------
  // Two ways of dealing the N atoms to the CTAs.  "Aligned": every unit is cut into k_u equal
  // parts, k_u = round(atoms_u / share), one part per CTA -- each CTA then touches one unit
  // only and a unit is merged from k_u records; chosen when the parts fit in one wave and the
  // largest exceeds the ideal share by no more than 24 atoms.  Otherwise "contiguous": the atoms of all units
  // laid end to end and cut into gridDim equal ranges, which balances any mix of list lengths
  // at the price of CTAs that straddle unit boundaries.
  N = sh.unit_start[U];
  if (tid < kCandidates) { sh.cand_parts[tid] = 0; sh.cand_max[tid] = 0; }
  if (tid == 0) sh.aligned = 0;
  __syncthreads();
  const bool try_aligned = (U <= kAlignedMaxUnits) && (N > 0);
  if (try_aligned && tid < U) {
    const int atoms = sh.unit_start[tid + 1] - sh.unit_start[tid];
    if (atoms > 0) {
#pragma unroll
      for (int c = 0; c < kCandidates; ++c) {
        // share_c = (N / G) * (1 + c / 16); 32-bit: atoms <= 12288, G ~ 148, N <= 2048 * 12288
        const unsigned int num = static_cast<unsigned int>(atoms) * G * 16u;
        const unsigned int den = static_cast<unsigned int>(N) * (16u + c);
        int k = static_cast<int>((2u * num + den) / (2u * den));  // round to nearest
        if (k < 1) k = 1;
        if (k > atoms) k = atoms;
        if (k * kMinPartAtoms > atoms) k = max(1, atoms / kMinPartAtoms);  // no part shorter than that
        if (P.pairs && k > 2 && atoms <= kPairAtoms) k = 2;  // short unit: two parts merge through shared memory
        atomicAdd(&sh.cand_parts[c], k);
        atomicMax(&sh.cand_max[c], (atoms + k - 1) / k);
      }
    }
  }
  __syncthreads();
  int cand = -1;
  if (try_aligned) {
    for (int c = 0; c < kCandidates; ++c)
      if (sh.cand_parts[c] <= G) { cand = c; break; }
    // worth it only while the parts stay close to the ideal share: a straddling CTA costs a
    // fixed few microseconds of extra merging, an oversized part costs time per atom
    if (cand >= 0 && static_cast<long long>(sh.cand_max[cand]) * G > N + 24ll * G) cand = -1;
  }
  aligned = cand >= 0;
  if (aligned && warp == 0) {  // first CTA of every unit: exclusive scan of k_u
    int carry = 0;
    for (int base = 0; base < U; base += 32) {
      const int u = base + lane;
      int k = 0;
      if (u < U) {
        const int atoms = sh.unit_start[u + 1] - sh.unit_start[u];
        if (atoms > 0) {
          const unsigned int num = static_cast<unsigned int>(atoms) * G * 16u;
          const unsigned int den = static_cast<unsigned int>(N) * (16u + cand);
          k = static_cast<int>((2u * num + den) / (2u * den));
          if (k < 1) k = 1;
          if (k > atoms) k = atoms;
        if (k * kMinPartAtoms > atoms) k = max(1, atoms / kMinPartAtoms);  // no part shorter than that
        if (P.pairs && k > 2 && atoms <= kPairAtoms) k = 2;  // short unit: two parts merge through shared memory
        }
      }
      int v = k;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += n;
      }
      if (u < U) sh.part_start[u + 1] = v + carry;
      if (base == 0 && lane == 0) sh.part_start[0] = 0;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  }
  __syncthreads();
  NP = aligned ? sh.part_start[U] : ((N < G) ? N : static_cast<long long>(G));
  }  // !planned
  if (warp < NC) {
    // consumers are the only writers of global memory: from here on the previous kernel's
    // results (and its use of the shared workspace) are complete
    if (P.lists_stable) pdl_wait();
    // units with an empty list: out = 0, lse = -inf
    for (int u = blockIdx.x; u < U; u += gridDim.x) {
      if (sh.unit_cnt[u] != 0) continue;
      const int b = u / P.Hkv, kvh = u % P.Hkv;
      for (int e = tid; e < P.M * kD; e += NC * 32) {
        const int r = e / kD, t = r / P.grp, h = kvh * P.grp + r % P.grp;
        P.out[((static_cast<long long>(b) * P.T + t) * P.Hq + h) * kD + e % kD] = 0.f;
        if (e % kD == 0) P.lse[(static_cast<long long>(b) * P.T + t) * P.Hq + h] = -INFINITY;
      }
    }
  }
  if (static_cast<long long>(blockIdx.x) >= NP) {
    if (paired) cluster_wait();
    return;
  }
  if (!planned) {
  if (aligned) {
    int lo = 0, hi = U - 1;  // unit whose CTA range holds this CTA
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (sh.part_start[mid] <= static_cast<int>(blockIdx.x)) lo = mid; else hi = mid - 1;
    }
    const int k = sh.part_start[lo + 1] - sh.part_start[lo];
    const int j = static_cast<int>(blockIdx.x) - sh.part_start[lo];
    const int atoms = sh.unit_start[lo + 1] - sh.unit_start[lo];  // j < k <= G: the products fit 32 bits
    a0 = sh.unit_start[lo] + j * atoms / k;
    a1 = sh.unit_start[lo] + (j + 1) * atoms / k;
  } else {
    a0 = cta_first_atom(blockIdx.x, N, NP);
    a1 = cta_first_atom(blockIdx.x + 1, N, NP);
  }

  // unit holding atom a0
  {
    int lo = 0, hi = U - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (sh.unit_start[mid] <= a0) lo = mid; else hi = mid - 1;
    }
    u_first = lo;
    while (sh.unit_start[u_first + 1] <= a0) ++u_first;  // skip empty units that share the start
  }
  }  // !planned

  if (warp >= NC) {
    // =========================== producer warps ===========================================
    const int pw = warp - NC;
    int it = 0, seg = 0;
    int last_it = -1;
    int a = a0, u = u_first;
    bool dead = false;
    while (a < a1 && !dead) {
      const int us = sh.unit_start[u], ue = sh.unit_start[u + 1];
      const int seg_hi = min(a1, ue);
      const int b = u / P.Hkv, kvh = u % P.Hkv;
      const int tok_lo = (a - us) * kAtom;
      const int tok_hi = min(sh.unit_cnt[u], (seg_hi - us) * kAtom);
      const int kvlen_b = P.kv_len[b];
      const int c_list = sh.unit_cnt[u] - P.tail;
      const int* list = P.dense ? nullptr
                                : P.idx + (static_cast<long long>(b) * P.G + ((P.G == 1) ? 0 : kvh)) * P.idx_stride;
      const __nv_bfloat16* kv_head = P.kv + static_cast<long long>(kvh) * P.s_head;
      // The query block of this unit (M rows of 256 bytes) is always fetched by producer warp
      // 0, walking the segments in order, so its parity wait can never be satisfied by a
      // stale phase.  For the first segment it goes out after the warp's first tile, so that
      // K/V prefetch is already in flight while the warp waits for the previous kernel.
      auto load_q = [&]() -> bool {
        if (seg == 0 && P.lists_stable) pdl_wait();
        if (kDirectQ && seg == 0) {
          // The consumers fetch the first query block themselves (see there); only the barrier's
          // phase is completed here, so that later segments find the parity they expect.  (No wait
          // on q_empty: nobody reads an older block, and the consumers may already have released
          // this one -- the "previous phase" a fresh barrier grants would then be one they hold.)
          if (lane == 0) mbar_arrive(&sh.q_full);
          return true;
        }
        if (!mbar_wait(&sh.q_empty, (seg & 1u) ^ 1u, &sh.abort_flag)) return false;
        if (lane == 0) mbar_arrive_expect_tx(&sh.q_full, static_cast<uint32_t>(P.M) * kRowBytes);
        __syncwarp();
        for (int r = lane; r < P.M; r += 32) {
          const int t = r / P.grp, h = kvh * P.grp + r % P.grp;
          bulk_g2s(sh.q + r * kPitch, P.q + ((static_cast<long long>(b) * P.T + t) * P.Hq + h) * kD,
                   kRowBytes, &sh.q_full);
        }
        return true;
      };
      bool q_pending = (pw == 0);
      if (q_pending && seg > 0) {
        q_pending = false;
        if (!load_q()) { sh.abort_flag = 1; dead = true; break; }
      }
      // lane j resolves tokens j and j + 32 of a tile to the byte offset of their K row:
      // list -> position -> block table -> page, two dependent loads, in two steps so that a
      // warp can keep the chain one tile of its own ahead (positions of its tile after next,
      // offsets of its next tile): neither load is then waited for between two tiles
      auto load_pos = [&](int t0, int (&pos)[2]) {
        const int ntok = min(kStageTok, tok_hi - t0);
#pragma unroll
        for (int jj = 0; jj < 2; ++jj) {
          const int k = t0 + min(lane + jj * 32, ntok - 1);  // token index inside the unit: the list first, then the tail
          pos[jj] = (k >= c_list) ? (kvlen_b + (k - c_list)) : (P.dense ? k : __ldg(list + k));
        }
      };
      auto offs_of = [&](const int (&posv)[2], long long (&off)[2]) -> bool {
        bool bad = false;
#pragma unroll
        for (int jj = 0; jj < 2; ++jj) {
          int pos = posv[jj];
          if (pos < 0 || pos >= kvlen_b + P.tail) { bad = true; pos = 0; }
          int lp = (P.page_shift >= 0) ? (pos >> P.page_shift) : (pos / P.page_size);
          // a position beyond the sequence's row of the block table (kv_len larger than the
          // table covers) is a bad index like any other: it reads position 0 instead
          if (lp >= P.bt_stride) { bad = true; pos = 0; lp = 0; }
          const int slot = pos - lp * P.page_size;
          long long page = P.bt ? static_cast<long long>(__ldg(P.bt + b * P.bt_stride + lp))
                                : (b * P.bt_stride + lp);
          if (page < 0 || (P.n_pages > 0 && page >= P.n_pages)) { bad = true; page = 0; }
          off[jj] = (page * P.s_page + static_cast<long long>(slot) * P.s_slot) * 2;
        }
        return bad;
      };
      auto resolve = [&](int t0, long long (&off)[2]) -> bool {
        int pos[2];
        load_pos(t0, pos);
        return offs_of(pos, off);
      };
      long long off_next[2] = {0, 0};
      bool bad_next = false;
      int t0_next = -1;  // tile whose offsets are already resolved
      int pos_nn[2] = {0, 0};
      int t0_nn = -1;    // tile whose positions are already loaded
      for (int t0 = tok_lo; t0 < tok_hi; t0 += kStageTok, ++it) {
        if ((it % kProdWarps) != pw) continue;
        const int s = it % kStages;
        const unsigned ph = (it / kStages) & 1u;
        long long off[2];
        bool bad;
        if (t0_next == t0) {
          off[0] = off_next[0];
          off[1] = off_next[1];
          bad = bad_next;
        } else {
          bad = resolve(t0, off);
        }
        if (!mbar_wait(&sh.empty[s], ph ^ 1u, &sh.abort_flag)) { sh.abort_flag = 1; dead = true; break; }
        const int ntok = min(kStageTok, tok_hi - t0);
        // The tail of a segment is padded to a whole 32-key block with copies of its last
        // token, so that every row a consumer multiplies by a zero weight holds finite data.
        const int npad = (ntok + 31) & ~31;
        // 16 lanes move one 256-byte row with 16-byte cp.async copies: a warp instruction
        // fetches two rows (four full 128-byte lines)
        const char* kbase = reinterpret_cast<const char*>(kv_head) + (lane & 15) * 16;
        const long long v_delta = P.s_kv * 2;
        const uint32_t k_dst = smem_u32(sh.kv[s][0]) + (lane >> 4) * kPitch + (lane & 15) * 16;
        const uint32_t v_dst = smem_u32(sh.kv[s][1]) + (lane >> 4) * kPitch + (lane & 15) * 16;
#pragma unroll
        for (int jj = 0; jj < 2; ++jj) {
#pragma unroll 4
          for (int i = 0; i < 16; ++i) {
            const int tok = jj * 32 + 2 * i + (lane >> 4);
            const long long o = __shfl_sync(0xffffffffu, off[jj], 2 * i + (lane >> 4));
            if (tok < npad) {
              cp_async16(k_dst + (jj * 32 + 2 * i) * kPitch, kbase + o);
              cp_async16(v_dst + (jj * 32 + 2 * i) * kPitch, kbase + o + v_delta);
            }
          }
        }
        // (test hook: the first tile of CTA 0 never completes, so the bounded waits run out)
        if (!(P.test_lose && blockIdx.x == 0 && it == 0)) cp_async_mbar_arrive_noinc(&sh.full[s]);
        if (q_pending) {
          q_pending = false;
          if (!load_q()) { sh.abort_flag = 1; dead = true; break; }
        }
        // Resolve this warp's next tile of the segment right after the copies went out (not
        // before: while the ring still has free slots the two dependent loads would delay
        // them by ~1.3 us), so that a slot's turnaround holds only the copy itself.
        t0_next = t0 + kProdWarps * kStageTok;
        if (t0_next < tok_hi) {
          if (t0_nn != t0_next) load_pos(t0_next, pos_nn);  // (first tile of the segment only)
          // positions of the tile after next first (independent), then the block-table loads
          int pos_new[2] = {0, 0};
          t0_nn = t0_next + kProdWarps * kStageTok;
          if (t0_nn < tok_hi) load_pos(t0_nn, pos_new); else t0_nn = -1;
          bad_next = offs_of(pos_nn, off_next);
          pos_nn[0] = pos_new[0];
          pos_nn[1] = pos_new[1];
        } else {
          t0_next = -1;
        }
        if (bad && P.status) atomicOr(P.status + b, SPECATTN_ROW_BAD_INDEX);
        last_it = it;
      }
      a = seg_hi;
      ++seg;
      if (a == ue) {
        ++u;
        while (u < U && sh.unit_start[u + 1] == sh.unit_start[u]) ++u;
      }
    }
    if (sh.abort_flag && last_it >= 0) {
      // give this warp's last copies a bounded chance to land before the CTA retires
      mbar_wait(&sh.full[last_it % kStages], (last_it / kStages) & 1u, nullptr);
    }
    if (paired) cluster_wait();
    return;
  }

  // =============================== consumer warps ===========================================
  const int mt = warp / WPM;            // 16-row slab of the query block
  const int wr = warp % WPM;            // role inside the slab
  // which tiles (it % 2) this warp reads.  Warps w and w + 4 share an SM sub-partition: they take
  // opposite parities, so that one is in its tensor phase while the other waits, exponentiates
  // or loads fragments (with equal parities both wait for the same tile and collide in every
  // phase: the tensor pipe was 47 % busy)
  const int parity = ((WPM == 4) ? (wr >> 1) : wr) ^ ((warp >> 2) & 1);
  const int g = lane >> 2, tq = lane & 3;
  const int lm = lane >> 3, lr = lane & 7;  // ldmatrix: matrix id, row within it
  const uint32_t q_addr = smem_u32(sh.q) + (mt * 16 + (lm & 1) * 8 + lr) * kPitch + (lm >> 1) * 16;
  // per-lane byte offsets inside a tile for the K (non-transposed) and V (transposed) fragments
  const uint32_t k_off = ((lm >> 1) * 8 + lr) * kPitch + (lm & 1) * 16;
  const uint32_t v_off = ((lm & 1) * 8 + lr) * kPitch + (lm >> 1) * 16;

  // A warp that meets a failed wait raises abort_flag and stops computing, but still walks
  // through the combine barriers of the segment it is in; every warp re-reads the flag right
  // after those barriers, so a whole slab group always leaves together.
  int it = 0, seg = 0;
  int a = a0, u = u_first;
  bool ok = true;
  bool peer_seen = false;
  constexpr bool kShareMerge = (WPM == 2);  // the slab's second warp helps with a final merge
  bool final_global = false;                // the CTA's last segment ends in a merge through global memory
  while (a < a1) {
    const int us = sh.unit_start[u], ue = sh.unit_start[u + 1];
    const int seg_hi = min(a1, ue);
    const int b = u / P.Hkv, kvh = u % P.Hkv;
    const int tok_lo = (a - us) * kAtom;
    const int tok_hi = min(sh.unit_cnt[u], (seg_hi - us) * kAtom);
    const int c_list = sh.unit_cnt[u] - P.tail;
    // in-flight tokens the two rows of this lane may see: row r belongs to query r / grp
    const int lim0 = (mt * 16 + g) / P.grp + P.tail_off;
    const int lim1 = (mt * 16 + g + 8) / P.grp + P.tail_off;

    // query fragments of this unit
    // With two warps per slab (query blocks of more than 32 rows) the query fragments are
    // re-read from shared memory for every block instead of being held in 32 registers: the
    // compiler spends those on fragment prefetch (dense, 40 rows: 3.11 -> 3.37 TB/s); with
    // four warps per slab the same change loses 3 %.
    uint32_t qf[8][4];
    if (kDirectQ && seg == 0) {
      // First query block of the CTA: every consumer warp copies the 16 rows of its own slab
      // itself (the warps of a slab write the same bytes), straight after its wait for
      // the previous kernel -- the queries are the one input that kernel may have produced.
      // Going through the producer warp (which first issues its K/V tile, then waits, then
      // starts a bulk copy) put ~2.5 us between the previous launch's end and the first product.
      for (int i = lane; i < 16 * 16; i += 32) {
        const int r = mt * 16 + (i >> 4), c = i & 15;
        if (r < P.M) {
          const int t = r / P.grp, h = kvh * P.grp + r % P.grp;
          cp_async16(smem_u32(sh.q) + r * kPitch + c * 16,
                     P.q + ((static_cast<long long>(b) * P.T + t) * P.Hq + h) * kD + c * 8);
        }
      }
      asm volatile("cp.async.wait_all;" ::: "memory");
      __syncwarp();
      ok = true;
    } else {
      ok = mbar_wait(&sh.q_full, seg & 1u, &sh.abort_flag);
    }
    if (!ok) sh.abort_flag = 1;
    if (!kQReload) {
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) ldmatrix_x4(qf[kk], q_addr + kk * 32);
      __syncwarp();
      if (ok && lane == 0) mbar_arrive(&sh.q_empty);
    }

    WarpState st;
#pragma unroll
    for (int n = 0; n < 16; ++n) st.acc[n][0] = st.acc[n][1] = st.acc[n][2] = st.acc[n][3] = 0.f;
    st.m0 = st.m1 = -INFINITY;
    st.l0 = st.l1 = 0.f;

    for (int t0 = tok_lo; ok && t0 < tok_hi; t0 += kStageTok, ++it) {
      if ((it & 1) != parity) continue;
      const int s = it % kStages;
      const unsigned ph = (it / kStages) & 1u;
      if (!mbar_wait(&sh.full[s], ph, &sh.abort_flag)) { sh.abort_flag = 1; ok = false; break; }
      const int ntok = min(kStageTok, tok_hi - t0);
      const uint32_t k_base = smem_u32(sh.kv[s][0]) + k_off;
      const uint32_t v_base = smem_u32(sh.kv[s][1]) + v_off;
      // index inside the tile of the first in-flight token (negative once the tile starts
      // inside the tail; out of reach when the call has no tail)
      const int tb = P.tail ? (c_list - t0) : (1 << 20);
      if (WPM == 4) {
        const int key0 = (wr & 1) * 32;
        if (key0 < ntok)
          attend_block32<kQReload>(st, qf, q_addr, k_base + key0 * kPitch, v_base + key0 * kPitch, ntok - key0, P.scale_log2, tq,
                         tb - key0, lim0, lim1);
      } else {
        attend_block32<kQReload>(st, qf, q_addr, k_base, v_base, ntok, P.scale_log2, tq, tb, lim0, lim1);
        if (32 < ntok)
          attend_block32<kQReload>(st, qf, q_addr, k_base + 32 * kPitch, v_base + 32 * kPitch, ntok - 32, P.scale_log2, tq,
                         tb - 32, lim0, lim1);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.empty[s]);
    }

    if (kQReload) {
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.q_empty);   // the query tile was read for the last time
    }
    // ---- end of the segment: row sums across the quad, then combine the slab's warps ---------
    if (paired && !peer_seen) {  // the peer's arrival at kernel start: long past by now
      cluster_wait();
      peer_seen = true;
    }
    float m0 = st.m0, m1 = st.m1, l0 = st.l0, l1 = st.l1;
    float (&acc)[16][4] = st.acc;
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
#pragma unroll
    for (int half = WPM / 2; half >= 1; half >>= 1) {
      if (wr >= half && wr < 2 * half) {
        // lane-major float4 records: 17 16-byte stores per lane
        float4* rec = reinterpret_cast<float4*>(sh.scratch[mt][wr - half]) + lane;
#pragma unroll
        for (int n = 0; n < 16; ++n) rec[n * 32] = make_float4(acc[n][0], acc[n][1], acc[n][2], acc[n][3]);
        rec[16 * 32] = make_float4(m0, l0, m1, l1);
      }
      named_bar_sync(1 + mt, WPM * 32);
      if (wr < half) {
        const float4* rec = reinterpret_cast<const float4*>(sh.scratch[mt][wr]) + lane;
        const float4 ml = rec[16 * 32];
        float mn, ao, ai;
        merge_scales(m0, ml.x, mn, ao, ai);
        l0 = l0 * ao + ml.y * ai;
        m0 = mn;
        float mn1, ao1, ai1;
        merge_scales(m1, ml.z, mn1, ao1, ai1);
        l1 = l1 * ao1 + ml.w * ai1;
        m1 = mn1;
#pragma unroll
        for (int n = 0; n < 16; ++n) {
          const float4 r = rec[n * 32];
          acc[n][0] = acc[n][0] * ao + r.x * ai;
          acc[n][1] = acc[n][1] * ao + r.y * ai;
          acc[n][2] = acc[n][2] * ao1 + r.z * ai1;
          acc[n][3] = acc[n][3] * ao1 + r.w * ai1;
        }
      }
      named_bar_sync(1 + mt, WPM * 32);
    }
    if (sh.abort_flag) { ok = false; break; }

    if (kShareMerge && seg_hi == a1 && !((a == us) && (seg_hi == ue))) final_global = true;
    if (wr == 0) {
      const bool whole = (a == us) && (seg_hi == ue);
      bool finish = whole;
      // A unit cut in exactly two parts whose CTAs form one cluster is merged through the even
      // CTA's shared memory: the odd CTA stores its record there and arrives on a barrier.
      const bool pair_merge = paired && aligned && !whole && (sh.part_start[u + 1] - sh.part_start[u] == 2) &&
                              ((sh.part_start[u] & 1) == 0);
      if (pair_merge) {
        if (cluster_cta_rank() == 1) {
          // 17 16-byte remote stores per lane (lane-major float4 records)
          const uint32_t dst = map_to_cta(smem_u32(sh.peer_rec[mt]), 0) + lane * 16;
#pragma unroll
          for (int n = 0; n < 16; ++n) st_cluster_v4(dst + n * 512, acc[n][0], acc[n][1], acc[n][2], acc[n][3]);
          st_cluster_v4(dst + 16 * 512, m0, l0, m1, l1);
          __syncwarp();
          if (lane == 0) mbar_arrive_remote(map_to_cta(smem_u32(&sh.peer_full), 0));
        } else {
          if (!mbar_wait_cluster(&sh.peer_full, 0u, &sh.abort_flag)) { sh.abort_flag = 1; ok = false; break; }
          const float4* rec = reinterpret_cast<const float4*>(sh.peer_rec[mt]) + lane;
          const float4 ml = rec[16 * 32];
          float mn, ao, ai;
          merge_scales(m0, ml.x, mn, ao, ai);
          l0 = l0 * ao + ml.y * ai;
          m0 = mn;
          float mn1, ao1, ai1;
          merge_scales(m1, ml.z, mn1, ao1, ai1);
          l1 = l1 * ao1 + ml.w * ai1;
          m1 = mn1;
#pragma unroll
          for (int n = 0; n < 16; ++n) {
            const float4 r = rec[n * 32];
            acc[n][0] = acc[n][0] * ao + r.x * ai;
            acc[n][1] = acc[n][1] * ao + r.y * ai;
            acc[n][2] = acc[n][2] * ao1 + r.z * ai1;
            acc[n][3] = acc[n][3] * ao1 + r.w * ai1;
          }
          finish = true;
        }
      } else if (!whole) {
        // publish this CTA's share of the unit, then see whether it was the last to arrive
        // lane-major float4 records, as in shared memory
        float4* rec = reinterpret_cast<float4*>(
                          P.partials + (static_cast<size_t>(2 * blockIdx.x + (a == a0 ? 0 : 1)) * MT + mt) * kRec) + lane;
#pragma unroll
        for (int n = 0; n < 16; ++n) __stcg(rec + n * 32, make_float4(acc[n][0], acc[n][1], acc[n][2], acc[n][3]));
        __stcg(rec + 16 * 32, make_float4(m0, l0, m1, l1));
        __threadfence();
        __syncwarp();
        const int i_lo = aligned ? sh.part_start[u] : cta_of_atom(us, N, NP);
        const int i_hi = aligned ? sh.part_start[u + 1] - 1 : cta_of_atom(ue - 1, N, NP);
        unsigned int old = 0;
        if (lane == 0) old = atomicAdd(P.counters + u * kCountersPerUnit + mt, 1u);
        old = __shfl_sync(0xffffffffu, old, 0);
        const bool last = old == static_cast<unsigned int>(i_hi - i_lo);
        if (kShareMerge && seg_hi == a1) {
          // final segment: the verdict goes to the slab's other warp; the merge follows the loop
          if (last) {
            __threadfence();
            if (lane == 0) {
              P.counters[u * kCountersPerUnit + mt] = 0u;  // ready for the next call
              sh.merge_arg[mt][0] = i_lo;
              sh.merge_arg[mt][1] = i_hi;
              sh.merge_arg[mt][2] = us;
              sh.merge_arg[mt][3] = b;
              sh.merge_arg[mt][4] = kvh;
            }
          }
          if (lane == 0) sh.merge_last[mt] = last ? 1 : 0;
        } else if (last) {
          finish = true;
          __threadfence();
          // Merge every contributor's record in CTA order (the own one included, read back
          // from memory, so the result does not depend on who arrived last).  First the
          // common maxima, then one scaled accumulation pass with independent loads.
          // (the loads of four records' maxima, then of two records' halves, are in flight together:
          // walking the records one round trip to L2 at a time took 6 - 8 us for four of them)
          auto record = [&](int i) -> const float4* {
            return reinterpret_cast<const float4*>(P.partials +
                (static_cast<size_t>(2 * i + ((aligned || cta_first_atom(i, N, NP) >= us) ? 0 : 1)) * MT + mt) * kRec) + lane;
          };
          m0 = m1 = -INFINITY;
          for (int i = i_lo; i <= i_hi; i += 4) {   // four records' maxima per round trip
            float4 ml[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) ml[j] = __ldcg(record(min(i + j, i_hi)) + 16 * 32);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              m0 = fmaxf(m0, ml[j].x);
              m1 = fmaxf(m1, ml[j].z);
            }
          }
          const float base0 = (m0 == -INFINITY) ? 0.f : m0, base1 = (m1 == -INFINITY) ? 0.f : m1;
          l0 = l1 = 0.f;
#pragma unroll
          for (int n = 0; n < 16; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            for (int i = i_lo; i <= i_hi; i += 2) {   // two records' half rows per round trip
              const bool two = i + 1 <= i_hi;
              const float4* ra = record(i);
              const float4* rb = record(two ? i + 1 : i);
              const float4 mla = __ldcg(ra + 16 * 32), mlb = __ldcg(rb + 16 * 32);
              float4 xa[8], xb[8];
#pragma unroll
              for (int n = 0; n < 8; ++n) {
                xa[n] = __ldcg(ra + (half * 8 + n) * 32);
                xb[n] = __ldcg(rb + (half * 8 + n) * 32);
              }
              const float wa0 = ex2(mla.x - base0), wa1 = ex2(mla.z - base1);
              const float wb0 = two ? ex2(mlb.x - base0) : 0.f, wb1 = two ? ex2(mlb.z - base1) : 0.f;
              if (half == 0) {
                l0 += mla.y * wa0;
                l1 += mla.w * wa1;
                if (two) {
                  l0 += mlb.y * wb0;
                  l1 += mlb.w * wb1;
                }
              }
#pragma unroll
              for (int n = 0; n < 8; ++n) {
                acc[half * 8 + n][0] += xa[n].x * wa0;
                acc[half * 8 + n][1] += xa[n].y * wa0;
                acc[half * 8 + n][2] += xa[n].z * wa1;
                acc[half * 8 + n][3] += xa[n].w * wa1;
                if (two) {
                  acc[half * 8 + n][0] += xb[n].x * wb0;
                  acc[half * 8 + n][1] += xb[n].y * wb0;
                  acc[half * 8 + n][2] += xb[n].z * wb1;
                  acc[half * 8 + n][3] += xb[n].w * wb1;
                }
              }
            }
          }
          if (lane == 0) P.counters[u * kCountersPerUnit + mt] = 0u;  // ready for the next call
        }
      }
      if (finish) {
        const float inv0 = (l0 > 0.f) ? 1.f / l0 : 0.f;
        const float inv1 = (l1 > 0.f) ? 1.f / l1 : 0.f;
        const int r0 = mt * 16 + g, r1 = r0 + 8;
        if (r0 < P.M) {
          const int t = r0 / P.grp, h = kvh * P.grp + r0 % P.grp;
          const long long row = (static_cast<long long>(b) * P.T + t) * P.Hq + h;
          float* o = P.out + row * kD + tq * 2;
#pragma unroll
          for (int n = 0; n < 16; ++n)
            *reinterpret_cast<float2*>(o + n * 8) = make_float2(acc[n][0] * inv0, acc[n][1] * inv0);
          if (tq == 0) P.lse[row] = (l0 > 0.f) ? (m0 + log2f(l0)) * kLn2 : -INFINITY;
        }
        if (r1 < P.M) {
          const int t = r1 / P.grp, h = kvh * P.grp + r1 % P.grp;
          const long long row = (static_cast<long long>(b) * P.T + t) * P.Hq + h;
          float* o = P.out + row * kD + tq * 2;
#pragma unroll
          for (int n = 0; n < 16; ++n)
            *reinterpret_cast<float2*>(o + n * 8) = make_float2(acc[n][2] * inv1, acc[n][3] * inv1);
          if (tq == 0) P.lse[row] = (l1 > 0.f) ? (m1 + log2f(l1)) * kLn2 : -INFINITY;
        }
      }
    }

    a = seg_hi;
    ++seg;
    if (a == ue) {
      ++u;
      while (u < U && sh.unit_start[u + 1] == sh.unit_start[u]) ++u;
    }
  }
  if (kShareMerge && final_global && ok) {
    // the CTA's last segment was one part of a cut unit: if this CTA arrived last there, each of
    // the slab's two warps merges half of the columns (after the loop: the verdict comes from
    // the first warp, and nothing of the unit's state is needed any more)
    named_bar_sync(1 + mt, WPM * 32);
    if (sh.merge_last[mt])
      merge_half<MT>(P, mt, wr, sh.merge_arg[mt][0], sh.merge_arg[mt][1], aligned, N, NP, sh.merge_arg[mt][2],
                     sh.merge_arg[mt][3], sh.merge_arg[mt][4]);
  }
  if (paired && !peer_seen) cluster_wait();
  if (!ok && P.status && lane == 0) atomicOr(P.status, SPECATTN_ROW_TIMEOUT);
}

template <int MT, int WPM>
cudaError_t launch(const VerifyParams& P, int n_ctas, cudaStream_t stream) {
  const size_t smem = sizeof(VShared<MT, WPM>) + 128;
  static std::atomic<unsigned long long> done_mask{0};  // per device: shared-memory opt-in done
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!((done_mask.load(std::memory_order_acquire) >> dev) & 1ull)) {
    err = cudaFuncSetAttribute(sparse_verify_kernel<MT, WPM>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               static_cast<int>(smem));
    if (err != cudaSuccess) return err;
    done_mask.fetch_or(1ull << dev, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(static_cast<unsigned>(n_ctas), 1, 1);
  cfg.blockDim = dim3((MT * WPM + kProdWarps) * 32, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (MT <= 2 && n_ctas % 2 == 0) {  // CTA pairs: short units are merged through peer shared memory
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  err = cudaLaunchKernelEx(&cfg, sparse_verify_kernel<MT, WPM>, P);
  if (err != cudaSuccess) cudaGetLastError();
  return err;
}

#include "sparse_verify_tc.cuh"

int m_tiles(const specattn_verify_args& A) {
  const int grp = A.n_q_heads / A.n_kv_heads;
  return (A.n_q * grp + 15) / 16;
}

int validate(const specattn_verify_args* args) {
  if (args == nullptr) return SPECATTN_ERR_NULL;
  if (args->struct_size != sizeof(specattn_verify_args)) return SPECATTN_ERR_STRUCT_SIZE;
  const specattn_verify_args& A = *args;
  if (A.batch < 0 || A.n_q < 1 || A.n_q_heads < 1 || A.n_kv_heads < 1 || A.page_size < 1 || A.n_groups < 1)
    return SPECATTN_ERR_RANGE;
  if (A.n_q_heads % A.n_kv_heads != 0) return SPECATTN_ERR_RANGE;
  if (A.n_groups != 1 && A.n_groups != A.n_kv_heads) return SPECATTN_ERR_RANGE;
  if (!(A.sm_scale >= 0.f)) return SPECATTN_ERR_RANGE;  // negative or NaN
  if (A.tail_len < 0 || A.tail_len > 64) return SPECATTN_ERR_RANGE;
  if ((A.flags & SPECATTN_VERIFY_ENGINE_MMA_SYNC) && (A.flags & SPECATTN_VERIFY_ENGINE_TCGEN05))
    return SPECATTN_ERR_RANGE;
  if (A.head_dim != kD) return SPECATTN_ERR_UNSUPPORTED;
  if (A.n_q * (A.n_q_heads / A.n_kv_heads) > SPECATTN_MAX_QUERY_ROWS) return SPECATTN_ERR_UNSUPPORTED;
  if (static_cast<long long>(A.batch) * A.n_kv_heads > kMaxUnits) return SPECATTN_ERR_UNSUPPORTED;
  return SPECATTN_OK;
}

// 32-row blocks of the query block (tcgen05 engine)
int row_blocks(const specattn_verify_args& A) { return (m_tiles(A) + 1) / 2; }

// Which engine runs a call: the caller's choice, else by what the host can see of the shape.
// Measured (dense, 32k-131k positions per sequence): with 33-64 query rows per KV head the
// mma.sync engine sits at its tensor-pipe ceiling (3.1-3.2 TB/s) and the tcgen05 engine reaches
// 3.6-3.9 TB/s; up to 32 rows, and on short lists at any size (one-shot set-up and merge cost),
// mma.sync is ahead.  List lengths live on the device, so only dense calls whose cache holds at
// least 8192 positions per sequence are switched.
bool page_granular(const specattn_verify_args& A);
bool use_tcgen05(const specattn_verify_args& A) {
  if (A.flags & SPECATTN_VERIFY_ENGINE_TCGEN05) return true;
  if (A.flags & SPECATTN_VERIFY_ENGINE_MMA_SYNC) return false;
  const long long rows = static_cast<long long>(A.n_q) * (A.n_q_heads / A.n_kv_heads);
  const long long capacity = static_cast<long long>(A.block_table_stride) * A.page_size;
  // (with page-wise K/V reads the tcgen05 engine is ahead on long dense caches at any number of
  // query rows: 24 rows over 4 x 131072 positions 5.5 TB/s against 5.3)
  return A.dense && capacity >= 8192 && (rows > 32 || page_granular(A));
}

// Page-granular K/V reads (tiled bulk tensor copies of 16-slot boxes) apply to dense calls and to
// lists the caller declares to be made of whole aligned 16-position chunks, when a page holds a
// multiple of 16 slots and the pool's extent is known.
bool page_granular(const specattn_verify_args& A) {
  return (A.dense || (A.flags & SPECATTN_VERIFY_PAGE_LISTS)) && A.page_size % 16 == 0 && A.n_pages > 0 &&
         A.n_pages < (1ll << 31) && A.n_kv_heads <= 256 && A.page_size <= 4096;
}

// The K/V pool as a 5-D tensor (element, head, slot, k/v, page) with a box of [64 elements x 1
// head x 16 slots], 128-byte swizzle: one box is one 128-byte half of 16 consecutive rows in the
// tcgen05 operand layout.  The driver's encoder is looked up through the runtime (no link-time
// dependency on the driver library).  Returns false if it is unavailable or refuses the strides.
bool make_kv_map(const specattn_verify_args& A, CUtensorMap* map) {
  typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static std::atomic<encode_fn> cached{nullptr};
  encode_fn fn = cached.load(std::memory_order_acquire);
  if (fn == nullptr) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || sym == nullptr) {
      cudaGetLastError();
      return false;
    }
    fn = reinterpret_cast<encode_fn>(sym);
    cached.store(fn, std::memory_order_release);
  }
  const cuuint64_t dims[5] = {static_cast<cuuint64_t>(kD), static_cast<cuuint64_t>(A.n_kv_heads),
                              static_cast<cuuint64_t>(A.page_size), 2ull, static_cast<cuuint64_t>(A.n_pages)};
  const cuuint64_t strides[4] = {static_cast<cuuint64_t>(A.stride_head) * 2, static_cast<cuuint64_t>(A.stride_slot) * 2,
                                 static_cast<cuuint64_t>(A.stride_kv) * 2, static_cast<cuuint64_t>(A.stride_page) * 2};
  const cuuint32_t box[5] = {64u, 1u, 16u, 1u, 1u};
  const cuuint32_t elem[5] = {1u, 1u, 1u, 1u, 1u};
  if (A.stride_head <= 0 || A.stride_slot <= 0 || A.stride_kv <= 0 || A.stride_page <= 0) return false;
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(A.kv_pages), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Sized for either engine, so that the choice never depends on the workspace at hand.
size_t workspace_bytes_for(const specattn_verify_args& A, int n_ctas) {
  const size_t a = static_cast<size_t>(m_tiles(A)) * kRec;
  const size_t b = static_cast<size_t>(row_blocks(A)) * kTcRec;
  return kCounterBytes + static_cast<size_t>(2) * n_ctas * (a > b ? a : b) * sizeof(float);
}

}  // namespace
}  // namespace specattn

using specattn::VerifyParams;

namespace specattn {
namespace {
// Pointer, alignment and stride rules of a call that will launch (everything except the
// workspace); shared by the entry points so that each of them checks before it enqueues anything.
int check_buffers(const specattn_verify_args& A) {
  if (!A.q || !A.kv_pages || !A.kv_len || !A.out || !A.lse) return SPECATTN_ERR_NULL;
  if (!A.dense && (!A.idx || !A.counts)) return SPECATTN_ERR_NULL;
  if (!A.dense && A.idx_stride < 0) return SPECATTN_ERR_RANGE;
  if (A.block_table_stride < 0 || A.n_pages < 0) return SPECATTN_ERR_RANGE;
  auto mis = [](const void* p, uintptr_t a) { return reinterpret_cast<uintptr_t>(p) % a != 0; };
  if (mis(A.q, 16) || mis(A.kv_pages, 16) || mis(A.out, 16)) return SPECATTN_ERR_ALIGN;
  if (A.stride_page % 8 || A.stride_kv % 8 || A.stride_slot % 8 || A.stride_head % 8) return SPECATTN_ERR_ALIGN;
  return SPECATTN_OK;
}

// The kernel-side view of the arguments (everything except the workspace).
VerifyParams make_params(const specattn_verify_args& A) {
  VerifyParams P;
  memset(&P, 0, sizeof(P));
  P.B = A.batch;
  P.T = A.n_q;
  P.Hq = A.n_q_heads;
  P.Hkv = A.n_kv_heads;
  P.grp = A.n_q_heads / A.n_kv_heads;
  P.M = P.T * P.grp;
  P.G = A.n_groups;
  P.dense = A.dense ? 1 : 0;
  P.page_size = A.page_size;
  P.page_shift = -1;
  for (int s = 0; s < 31; ++s)
    if ((1 << s) == A.page_size) P.page_shift = s;
  P.q = static_cast<const __nv_bfloat16*>(A.q);
  P.kv = static_cast<const __nv_bfloat16*>(A.kv_pages);
  P.n_pages = A.n_pages;
  P.s_page = A.stride_page;
  P.s_kv = A.stride_kv;
  P.s_slot = A.stride_slot;
  P.s_head = A.stride_head;
  P.bt = A.block_table;
  P.bt_stride = A.block_table_stride;
  P.kv_len = A.kv_len;
  P.idx = A.idx;
  P.idx_stride = A.idx_stride;
  P.counts = A.counts;
  const float scale = (A.sm_scale != 0.f) ? A.sm_scale : 1.0f / sqrtf(static_cast<float>(A.head_dim));
  P.scale_log2 = scale * specattn::kLog2e;
  P.out = A.out;
  P.lse = A.lse;
  P.status = A.status;
  P.lists_stable = (A.flags & SPECATTN_VERIFY_LISTS_STABLE) ? 1 : 0;
  P.tail = A.tail_len;
  P.tail_off = A.tail_len - A.n_q;

  P.plan = static_cast<const int*>(A.plan);
  P.test_lose = (A.flags & SPECATTN_VERIFY_TEST_LOSE_ARRIVAL) ? 1 : 0;
  P.pairs = (m_tiles(A) <= 2 && device_sm_count() % 2 == 0) ? 1 : 0;  // as launch() decides
  return P;
}
}  // namespace
}  // namespace specattn


extern "C" size_t specattn_verify_workspace_bytes(const specattn_verify_args* args) {
  if (specattn::validate(args) != SPECATTN_OK) return 0;
  const int n = specattn::device_sm_count();
  if (n <= 0) return 0;
  return specattn::workspace_bytes_for(*args, n);
}

extern "C" int specattn_verify_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (workspace == nullptr) return SPECATTN_ERR_NULL;
  if (workspace_bytes < specattn::kCounterBytes) return SPECATTN_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return SPECATTN_ERR_ALIGN;
  if (cudaMemsetAsync(workspace, 0, specattn::kCounterBytes, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
    cudaGetLastError();
    return SPECATTN_ERR_CUDA;
  }
  return SPECATTN_OK;
}

extern "C" int specattn_sparse_verify(const specattn_verify_args* args, void* cuda_stream) {
  specattn::NvtxRange nvtx_range("specattn_sparse_verify");
  const int v = specattn::validate(args);
  if (v != SPECATTN_OK) return v;
  const specattn_verify_args& A = *args;
  if (A.batch == 0) return SPECATTN_OK;
  const int pc = specattn::check_buffers(A);
  if (pc != SPECATTN_OK) return pc;
  if (!A.workspace) return SPECATTN_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(A.workspace) % 256 != 0) return SPECATTN_ERR_ALIGN;
  const int n_ctas = specattn::device_sm_count();
  if (n_ctas <= 0) return SPECATTN_ERR_CUDA;
  if (A.workspace_bytes < specattn::workspace_bytes_for(A, n_ctas)) return SPECATTN_ERR_WORKSPACE;

  VerifyParams P = specattn::make_params(A);
  P.counters = static_cast<unsigned int*>(A.workspace);
  P.partials = reinterpret_cast<float*>(static_cast<unsigned char*>(A.workspace) + specattn::kCounterBytes);

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t err;
  if (specattn::use_tcgen05(A)) {
    alignas(64) CUtensorMap kv_map;
    memset(&kv_map, 0, sizeof(kv_map));
    if (specattn::page_granular(A) && specattn::make_kv_map(A, &kv_map)) {
      switch (specattn::m_tiles(A)) {
        case 1: err = specattn::launch_tc<1, true>(P, kv_map, n_ctas, stream); break;
        case 2: err = specattn::launch_tc<2, true>(P, kv_map, n_ctas, stream); break;
        case 3: err = specattn::launch_tc<3, true>(P, kv_map, n_ctas, stream); break;
        default: err = specattn::launch_tc<4, true>(P, kv_map, n_ctas, stream); break;
      }
    } else {
      switch (specattn::m_tiles(A)) {
        case 1: err = specattn::launch_tc<1, false>(P, kv_map, n_ctas, stream); break;
        case 2: err = specattn::launch_tc<2, false>(P, kv_map, n_ctas, stream); break;
        case 3: err = specattn::launch_tc<3, false>(P, kv_map, n_ctas, stream); break;
        default: err = specattn::launch_tc<4, false>(P, kv_map, n_ctas, stream); break;
      }
    }
  } else {
    switch (specattn::m_tiles(A)) {
      case 1: err = specattn::launch<1, 4>(P, n_ctas, stream); break;
      case 2: err = specattn::launch<2, 4>(P, n_ctas, stream); break;
      case 3: err = specattn::launch<3, 2>(P, n_ctas, stream); break;
      default: err = specattn::launch<4, 2>(P, n_ctas, stream); break;
    }
  }
  if (err != cudaSuccess) return SPECATTN_ERR_CUDA;
  specattn::g_launch_count.fetch_add(1, std::memory_order_relaxed);
  return SPECATTN_OK;
}

extern "C" size_t specattn_verify_plan_bytes(const specattn_verify_args* args) {
  if (specattn::validate(args) != SPECATTN_OK) return 0;
  const int n = specattn::device_sm_count();
  if (n <= 0) return 0;
  return specattn::plan_ints(args->batch * args->n_kv_heads, n) * sizeof(int);
}

extern "C" int specattn_verify_plan(const specattn_verify_args* args, void* plan, size_t plan_bytes,
                                    void* cuda_stream) {
  specattn::NvtxRange nvtx_range("specattn_verify_plan");
  const int v = specattn::validate(args);
  if (v != SPECATTN_OK) return v;
  const specattn_verify_args& A = *args;
  if (plan == nullptr || !A.kv_len) return SPECATTN_ERR_NULL;
  if (!A.dense && !A.counts) return SPECATTN_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(plan) % 16 != 0) return SPECATTN_ERR_ALIGN;
  const int n_ctas = specattn::device_sm_count();
  if (n_ctas <= 0) return SPECATTN_ERR_CUDA;
  if (plan_bytes < specattn::plan_ints(A.batch * A.n_kv_heads, n_ctas) * sizeof(int)) return SPECATTN_ERR_WORKSPACE;
  if (A.batch == 0) return SPECATTN_OK;
  VerifyParams P = specattn::make_params(A);
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(1, 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = static_cast<cudaStream_t>(cuda_stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, specattn::verify_plan_kernel, P, static_cast<int*>(plan), n_ctas) != cudaSuccess) {
    cudaGetLastError();
    return SPECATTN_ERR_CUDA;
  }
  specattn::g_launch_count.fetch_add(1, std::memory_order_relaxed);
  return SPECATTN_OK;
}

extern "C" int specattn_verify_plan_many(const specattn_verify_args* const* args, void* const* plans,
                                         const size_t* plan_bytes, int32_t n, void* cuda_stream) {
  specattn::NvtxRange nvtx_range("specattn_verify_plan_many");
  if (n < 0) return SPECATTN_ERR_RANGE;
  if (n == 0) return SPECATTN_OK;
  if (args == nullptr || plans == nullptr || plan_bytes == nullptr) return SPECATTN_ERR_NULL;
  const int n_ctas = specattn::device_sm_count();
  if (n_ctas <= 0) return SPECATTN_ERR_CUDA;
  for (int i = 0; i < n; ++i) {  // everything is checked before anything is launched
    const int v = specattn::validate(args[i]);
    if (v != SPECATTN_OK) return v;
    const specattn_verify_args& A = *args[i];
    if (plans[i] == nullptr || !A.kv_len) return SPECATTN_ERR_NULL;
    if (!A.dense && !A.counts) return SPECATTN_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(plans[i]) % 16 != 0) return SPECATTN_ERR_ALIGN;
    if (plan_bytes[i] < specattn::plan_ints(A.batch * A.n_kv_heads, n_ctas) * sizeof(int)) return SPECATTN_ERR_WORKSPACE;
  }
  for (int i0 = 0; i0 < n; i0 += specattn::kPlanBatch) {
    specattn::PlanBatch B;
    memset(&B, 0, sizeof(B));
    int m = 0;
    for (int i = i0; i < n && i < i0 + specattn::kPlanBatch; ++i) {
      if (args[i]->batch == 0) continue;
      B.p[m] = specattn::make_params(*args[i]);
      B.plan[m] = static_cast<int*>(plans[i]);
      ++m;
    }
    if (m == 0) continue;
    B.G = n_ctas;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(static_cast<unsigned>(m), 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.stream = static_cast<cudaStream_t>(cuda_stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, specattn::verify_plan_many_kernel, B) != cudaSuccess) {
      cudaGetLastError();
      return SPECATTN_ERR_CUDA;
    }
    specattn::g_launch_count.fetch_add(1, std::memory_order_relaxed);
  }
  return SPECATTN_OK;
}

// ---------------------------------------------------------------------------------------------
// The variant for callers that cannot allocate: scratch lives in this library image.
namespace specattn {
namespace {
// One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[SPECATTN_STATIC_SCRATCH_BYTES];
}  // namespace
}  // namespace specattn

extern "C" int specattn_sparse_verify_static(const specattn_verify_args* args, void* cuda_stream) {
  const int v = specattn::validate(args);
  if (v != SPECATTN_OK) return v;
  if (args->batch == 0) return SPECATTN_OK;
  // every argument check comes before the first thing that is enqueued
  const int pc = specattn::check_buffers(*args);
  if (pc != SPECATTN_OK) return pc;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return SPECATTN_ERR_CUDA;
  }
  const int n_ctas = specattn::device_sm_count();
  if (n_ctas <= 0) return SPECATTN_ERR_CUDA;
  if (specattn::workspace_bytes_for(*args, n_ctas) > SPECATTN_STATIC_SCRATCH_BYTES)
    return SPECATTN_ERR_STATIC_SCRATCH;
  // In host code the array's name is only a handle; the kernel needs its device address,
  // looked up once per device with that device current (racing first callers store the same
  // value).
  static std::atomic<void*> device_addr[64];
  void* scratch = device_addr[dev].load(std::memory_order_acquire);
  if (scratch == nullptr) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, specattn::g_static_scratch);
    if (e != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return SPECATTN_ERR_CUDA;
    }
    device_addr[dev].store(p, std::memory_order_release);
    scratch = p;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // the array keeps the previous call's contents: the arrival counters must start at zero
  if (cudaMemsetAsync(scratch, 0, specattn::kCounterBytes, stream) != cudaSuccess) {
    cudaGetLastError();
    return SPECATTN_ERR_CUDA;
  }
  specattn_verify_args a = *args;
  a.workspace = scratch;
  a.workspace_bytes = SPECATTN_STATIC_SCRATCH_BYTES;
  return specattn_sparse_verify(&a, cuda_stream);
}
