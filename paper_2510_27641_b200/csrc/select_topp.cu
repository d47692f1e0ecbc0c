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
//   2. builds the level-1 histogram of mantissa sums in shared memory: all values of a bin
//      share one exponent, so the sum of their 24-bit mantissas is an exact integer and the
//      result does not depend on the order of the updates.  The sum is kept as two 32-bit
//      words (low 16 and high 8 mantissa bits), each updated with a fire-and-forget 32-bit
//      reduction, so consecutive updates pipeline.  Warps whose lanes all hit one bin (ties,
//      the common case for attention rows) pre-reduce with redux.sync first.
//   3. the histograms are reduced across the cluster through distributed shared memory: at
//      level 1 each CTA owns a bin range and all gather the result; at levels 2 and 3 (only
//      the elements inside the threshold bin) every CTA reads all peers' histograms itself.
//      Every CTA scans the reduced bins with the same warp-shuffle suffix scan in binary64,
//      so all arrive at the same bin without a broadcast.  (Remote atomics into one CTA's
//      histogram were measured first and cost ~11 us per level on tie-free rows.)
//      When the level-1 threshold bin holds at most 512 values (its exact mantissa sum bounds
//      their number) levels 2 and 3 are replaced by a short cut: every CTA collects its keys of
//      that bin, all CTAs fetch all of them and pick the threshold key directly.
//   4. after three levels the threshold is known bit-exactly; each CTA compacts its kept
//      positions in ascending order behind the counts of the lower-ranked CTAs.
// When a list has a single contributing row (one draft head, gamma = 1: the selection
// micro-benchmark) of 32k positions or more there is nothing to aggregate and the row is not
// copied to shared memory at all but re-read from global memory (L2) by the later passes,
// which shrinks a CTA to ~51 KB of shared memory so that four of them share an SM.
// With a workspace and few lists the call becomes two launches: aggregate_rows_kernel sums the
// rows with 512 positions per CTA (the whole GPU streams, however few the lists) and the
// search runs in place over that sum.
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <float.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#include <atomic>

#include "ptx.cuh"
#include "nvtx_range.h"
#include "specattn.h"

namespace cg = cooperative_groups;

namespace specattn {

extern std::atomic<long long> g_launch_count;

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kChunk = 2048;             // positions per staged row piece (8 KB)
constexpr int kDepth = 8;                // row pieces in flight per thread (ring of 8 x 8 KB)
constexpr int kL1Bins = 2048;            // sign(0) + 8 exponent bits + 3 mantissa bits
constexpr int kL23Bins = 1024;           // 10 mantissa bits per later level
constexpr int kGroup = 32;               // bins per scan group (one warp-wide scan)
constexpr int kSliceCap = 24576;         // positions per CTA
constexpr unsigned int kFull = 0xffffffffu;
constexpr int kDirectMax = 128;         // up to this many gathered keys the threshold is searched directly
constexpr int kCandCap = 512;           // keys of the threshold bin that the short cut below can hold

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
  int single_row;  // every list has exactly one contributing row: read it in place
  int per_step;    // Alg. 2 as printed: one nucleus per speculated query, unioned
  int bisect_iters;  // > 0: the threshold is the last midpoint of that many bisection steps
  int chunk;         // > 1: selection over per-chunk sums (power of two, 4..64); kept chunks keep all positions
  const float* agg;  // two-launch form: the aggregated rows, [list][L_stride], written by aggregate_rows_kernel
};

// A histogram of exact mantissa sums, kept as two 32-bit words: `lo` sums the low 16 mantissa
// bits, `hi` the high 8 (a slice holds < 2^15 elements, so neither can wrap) and the total is
// (hi << 16) + lo.  Updates never read a value back.  A bin is empty iff its sum is zero (zeros
// are never entered, every other value has a non-zero mantissa).
struct Hist {
  unsigned int* lo;
  unsigned int* hi;
};

struct Shared {
  unsigned int h_lo[kL1Bins];  // level-1 histogram of this CTA
  unsigned int h_hi[kL1Bins];
  double grp_mass[kL1Bins / kGroup];
  int warp_cnt[kWarps];
  int n_rows;
  int n_invalid;            // threads of this CTA that met an invalid input
  float warp_max[kWarps];   // largest aggregated value seen by each warp (literal bisection only)
  float cta_max;            // read by the other CTAs of the cluster
  int local_kept;           // read by the other CTAs of the cluster
  int bin_lo, bin_hi;       // first and last non-empty level-1 bin of this CTA (read by the cluster)
  unsigned int bin_kmin, bin_kmax;  // (rows read in place) smallest / largest key of this CTA inside the
                                    // level-1 threshold bin (read by the cluster)
  int n_cand;               // keys this CTA found in the level-1 threshold bin (read by the cluster)
  unsigned int cand[kCandCap];
  int cand_pos[kCandCap];   // (rows read in place) their positions inside the slice
  unsigned int all_keys[kCandCap];  // the keys of the whole cluster in that bin (short cut)
  unsigned int red_key[2 * kWarps];
  unsigned long long red_sum[2 * kWarps];
  // result of a scan (written by warp 0)
  int found_bin;
  double mass_above;        // mass strictly above the found bin (incl. carry)
  double mass_ge;           // mass_above + mass of the found bin
  double total;             // mass of everything at this level plus the carry
};

// Layout of the dynamic shared memory behind `Shared`: the aggregated slice, then the staging
// ring.  Once the slice is aggregated the ring is idle and hosts
//   [0, 16 KB)   reduced bin masses (binary64), read by the level scans
//   [16, 24 KB)  level-2 histogram of this CTA (low and high words)
//   [24, 32 KB)  level-3 histogram of this CTA
constexpr int kRingFloats = kDepth * kChunk;
// a list read in place needs the fixed part and 32 KB of scan arrays: four such CTAs (plus 1 KB
// each that the system reserves) must fit the 227 KB of an SM
static_assert(4 * (((sizeof(Shared) + 127) / 128) * 128 + 32 * 1024 + 1024) <= 227 * 1024,
              "four in-place CTAs per SM");
static_assert(kRingFloats * 4 >= 32 * 1024, "the ring must hold the scan arrays");

__device__ __forceinline__ double pow2_double(int k) {  // 2^k, k in the normal range
  return __longlong_as_double(static_cast<long long>(k + 1023) << 52);
}

__device__ __forceinline__ unsigned int mantissa_of(unsigned int key) {
  return (key >> 23) ? ((key & 0x7fffffu) | 0x800000u) : (key & 0x7fffffu);
}

__device__ __forceinline__ void hist_bump(const Hist& h, int bin, unsigned int lo, unsigned int hi) {
  atomicAdd(&h.lo[bin], lo);
  atomicAdd(&h.hi[bin], hi);
}

// Adds one value to a histogram bin (all 32 lanes call this together).  When every taking
// lane hits the same bin the warp pre-reduces and one lane issues the atomic.
__device__ __forceinline__ void hist_add(const Hist& h, bool take, int bin, unsigned int mant) {
  const unsigned takers = __ballot_sync(kFull, take);
  if (takers == 0) return;
  const int leader = __ffs(takers) - 1;
  const int lead_bin = __shfl_sync(kFull, bin, leader);
  const bool same = __all_sync(kFull, !take || bin == lead_bin);
  if (same && __popc(takers) > 1) {
    const unsigned int slo = __reduce_add_sync(kFull, take ? (mant & 0xffffu) : 0u);
    const unsigned int shi = __reduce_add_sync(kFull, take ? (mant >> 16) : 0u);
    if ((threadIdx.x & 31) == leader) hist_bump(h, lead_bin, slo, shi);
  } else if (take) {
    hist_bump(h, bin, mant & 0xffffu, mant >> 16);
  }
}

// The four values of a lane's float4 at once: one uniformity test per 128 values instead of one
// per 32 (the test costs more than the update it saves unless whole warps tie).
__device__ __forceinline__ void hist_add4(const Hist& h, const bool (&take)[4], const int (&bin)[4],
                                          const unsigned int (&mant)[4]) {
  const bool any = take[0] || take[1] || take[2] || take[3];
  const unsigned takers = __ballot_sync(kFull, any);
  if (takers == 0) return;
  const int leader = __ffs(takers) - 1;
  const int my_first = take[0] ? bin[0] : take[1] ? bin[1] : take[2] ? bin[2] : bin[3];
  const int lead_bin = __shfl_sync(kFull, my_first, leader);
  bool mine_same = true;
#pragma unroll
  for (int e = 0; e < 4; ++e) mine_same = mine_same && (!take[e] || bin[e] == lead_bin);
  if (__all_sync(kFull, mine_same)) {
    unsigned int lo = 0u, hi = 0u;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      lo += take[e] ? (mant[e] & 0xffffu) : 0u;
      hi += take[e] ? (mant[e] >> 16) : 0u;
    }
    const unsigned int slo = __reduce_add_sync(kFull, lo);
    const unsigned int shi = __reduce_add_sync(kFull, hi);
    if ((threadIdx.x & 31) == leader) hist_bump(h, lead_bin, slo, shi);
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (take[e]) hist_bump(h, bin[e], mant[e] & 0xffffu, mant[e] >> 16);
  }
}

// Appends the keys of the taking lanes to the CTA's candidate list (all 32 lanes call this
// together); slots beyond the capacity are counted but not stored.
__device__ __forceinline__ void cand_add(Shared& sh, bool take, unsigned int key, int pos) {
  const unsigned takers = __ballot_sync(kFull, take);
  if (takers == 0) return;
  const int lane = threadIdx.x & 31;
  const int leader = __ffs(takers) - 1;
  int base = 0;
  if (lane == leader) base = atomicAdd(&sh.n_cand, __popc(takers));
  base = __shfl_sync(kFull, base, leader);
  const int slot = base + __popc(takers & ((1u << lane) - 1u));
  if (take && slot < kCandCap) {
    sh.cand[slot] = key;
    sh.cand_pos[slot] = pos;
  }
}

__device__ __forceinline__ double shfl_down_f64(double v, int d) { return __shfl_down_sync(kFull, v, d); }

// Scan of `nbins` reduced bins (nbins = 32 * groups, groups <= 64): finds the highest bin at
// which the mass accumulated from the top -- starting from `carry_mass` already above this
// level -- reaches `target` (or p * everything when `target_is_fraction`).  All sums run in
// one fixed order (per-group serial sums, then shuffle suffix scans in warp 0), so every CTA
// of a cluster gets bit-identical results.  Results land in sh.found_bin, sh.mass_above,
// sh.mass_ge, sh.total.  Called by all threads.  An empty bin has mass exactly 0.
__device__ void scan_bins(Shared& sh, const double* mass, int nbins, double carry_mass, double target,
                          bool target_is_fraction, float p, int grp_lo = 0, int grp_hi = 1 << 20) {
  const int groups = nbins / kGroup;
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  // group sums: four threads per group add eight bins each (top bin first), then combine; the
  // order is fixed, and consecutive threads read consecutive 64-byte pieces (a thread per group
  // walking its 256 bytes put all lanes of a warp on one bank)
  {
    const int grp = tid >> 2, part = tid & 3;
    double s = 0.0;
    if (grp < groups && grp >= grp_lo && grp < grp_hi) {  // groups outside the range are empty and unwritten
      const double* m8 = mass + grp * kGroup + part * 8;
#pragma unroll
      for (int b = 7; b >= 0; --b) s += m8[b];
    }
    const double s1 = s + __shfl_xor_sync(kFull, s, 1);      // (0+1), (2+3)
    const double s2 = s1 + __shfl_xor_sync(kFull, s1, 2);    // all four quarters
    if (grp < groups && part == 0) sh.grp_mass[grp] = s2;
  }
  __syncthreads();
  if (tid < 32) {
    // lane l owns groups 2l (low) and 2l+1 (high) when there are 64 groups, group l otherwise
    const bool two = groups > 32;
    const double g_hi = two ? sh.grp_mass[2 * lane + 1] : sh.grp_mass[lane];
    const double g_lo = two ? sh.grp_mass[2 * lane] : 0.0;
    // inclusive suffix sums over lanes (lane 31 holds the top groups)
    double s = g_hi + g_lo;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const double sv = shfl_down_f64(s, d);
      if (lane + d < 32) s += sv;
    }
    // mass of everything strictly above this lane's groups, plus the carry
    double above = shfl_down_f64(s, 1);
    if (lane == 31) above = 0.0;
    above += carry_mass;
    const double all = __shfl_sync(kFull, s, 0) + carry_mass;
    if (target_is_fraction) target = static_cast<double>(p) * all;
    // suffix mass including the high group, and including both
    const double with_hi = above + g_hi;
    const double with_lo = with_hi + g_lo;
    // highest non-empty group whose inclusive suffix reaches the target
    const bool hit_hi = (g_hi != 0.0) && (with_hi >= target);
    const bool hit_lo = two && (g_lo != 0.0) && (with_lo >= target);
    const unsigned hits = __ballot_sync(kFull, hit_hi || hit_lo);
    int grp;            // chosen group
    int src;            // lane that owns it
    bool pick_hi;
    if (hits != 0u) {
      src = 31 - __clz(hits);
      pick_hi = __shfl_sync(kFull, hit_hi ? 1 : 0, src) != 0;
      grp = two ? (2 * src + (pick_hi ? 1 : 0)) : src;
    } else {
      // only reachable through rounding between two summation orders: take the lowest
      // non-empty group, i.e. everything at this level is kept
      const unsigned ne_lo = __ballot_sync(kFull, two ? (g_lo != 0.0) : (g_hi != 0.0));
      const unsigned ne_hi = __ballot_sync(kFull, two && (g_hi != 0.0));
      int g0 = -1;
      for (int l = 0; l < 32 && g0 < 0; ++l) {
        if (two) {
          if ((ne_lo >> l) & 1u) g0 = 2 * l;
          else if ((ne_hi >> l) & 1u) g0 = 2 * l + 1;
        } else if ((ne_lo >> l) & 1u) {
          g0 = l;
        }
      }
      if (g0 < 0) g0 = 0;
      grp = g0;
      src = two ? (g0 >> 1) : g0;
      pick_hi = two ? ((g0 & 1) != 0) : true;
    }
    // mass strictly above the chosen group (incl. carry)
    const double b_hi = __shfl_sync(kFull, above, src), b_lo = __shfl_sync(kFull, with_hi, src);
    const double base = pick_hi ? b_hi : b_lo;
    // inside the group: lane b <-> bin grp * 32 + b, inclusive suffix over lanes
    const double m = mass[grp * kGroup + lane];
    double si = m;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const double sv = shfl_down_f64(si, d);
      if (lane + d < 32) si += sv;
    }
    const double incl = base + si;  // mass of bins >= this one (incl. carry)
    double ab = shfl_down_f64(si, 1);
    if (lane == 31) ab = 0.0;
    const unsigned ok = __ballot_sync(kFull, m != 0.0 && incl >= target);
    const unsigned nonempty = __ballot_sync(kFull, m != 0.0);
    int fb;
    if (ok != 0u) fb = 31 - __clz(ok);
    else if (nonempty != 0u) fb = __ffs(nonempty) - 1;  // rounding: keep the whole group
    else fb = 0;
    const double f_above = base + __shfl_sync(kFull, ab, fb);
    const double f_ge = __shfl_sync(kFull, incl, fb);
    if (lane == 0) {
      sh.found_bin = grp * kGroup + fb;
      sh.mass_above = f_above;
      sh.mass_ge = f_ge;
      sh.total = all;
    }
  }
  __syncthreads();
}

// kVariant: the selection variants of Alg. 2 (per-step union, fixed-iteration bisection); the
// default instantiation contains none of their code.
template <bool kInPlace, bool kVariant>
__global__ void __launch_bounds__(kThreads, kInPlace ? 4 : 2) select_topp_kernel(const __grid_constant__ SelectParams P) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Shared& sh = *reinterpret_cast<Shared*>(smem_raw);
  // behind the fixed part: the element offset of each contributing row, in add order (a row
  // read in place is its list's only row, at offset 0, and has no such table), then the slice
  long long* const row_off = reinterpret_cast<long long*>(smem_raw + ((sizeof(Shared) + 127) / 128) * 128);
  float* a = reinterpret_cast<float*>(smem_raw + ((sizeof(Shared) + 127) / 128) * 128 +
                                      (kInPlace ? 0 : SPECATTN_MAX_ROWS_PER_LIST * sizeof(long long)));

  cg::cluster_group cluster = cg::this_cluster();
  const int cs = static_cast<int>(cluster.num_blocks());
  const int rank = static_cast<int>(cluster.block_rank());
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  // a one-CTA "cluster" needs no hardware cluster barrier (~0.7 us each, seven per list)
  auto csync = [&]() {
    if (cs > 1) cluster.sync(); else __syncthreads();
  };

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
  const int align = (kVariant && P.chunk > 4) ? P.chunk : 4;  // slices start on 16 bytes and on a chunk
  const int per = ((L + cs - 1) / cs + align - 1) & ~(align - 1);
  const int lo = min(L, rank * per);
  const int hi = min(L, lo + per);
  const int n_loc = hi - lo;

  // dynamic shared memory behind the fixed part
  const int slice_cap = kInPlace ? 0 : static_cast<int>(((((P.L_stride + cs - 1) / cs + align - 1) & ~static_cast<long long>(align - 1)) + 31) & ~31ll);
  float* ring = a + slice_cap;
  double* const r_mass = reinterpret_cast<double*>(ring);
  unsigned int* const lvl_base = reinterpret_cast<unsigned int*>(ring + 4096);  // 2 levels x (lo, hi) x 1024
  const Hist h1 = {sh.h_lo, sh.h_hi};

  const float* A = (kInPlace && P.agg != nullptr)
                       ? P.agg + static_cast<long long>(list) * P.L_stride + lo
                       : P.probs[slot] + static_cast<long long>(b) * P.H * P.gamma * P.L_stride + lo;
  constexpr bool in_place = kInPlace;
  // bit pattern of aggregated position i of the slice (-0.0 reads as +0.0)
  auto key_at = [&](int i) -> unsigned int {
    return in_place ? __float_as_uint(__ldg(A + i) + 0.f) : __float_as_uint(a[i]);
  };
  const int n4 = (n_loc + 3) >> 2;
  // (rows read in place) float4s in whole iterations of the CTA whose values all lie inside the
  // slice: the lean bodies of the passes cover [0, n4_main), the general ones the rest
  const int n4_main = ((n_loc >> 2) / (4 * kThreads)) * (4 * kThreads);
  // In-place passes read the row from global memory (L2) with four independent 16-byte loads per
  // thread in flight: with one dependent load per iteration a CTA moved ~4 GB/s (latency-bound);
  // eight in flight were 3-4 % slower on 64k / 128k rows than four (twice the code per pass), two
  // 3 % slower again.  Asking for the pieces ahead into L2 (bulk prefetch, 64 KB ahead per CTA)
  // changed nothing: the passes are not waiting for HBM.  Two copies of the level-1 histogram for
  // even and odd lanes (rows of probabilities only use the lower half of the bins) made the pass
  // 30 % slower, with the copies in the same banks or in different ones: lanes that hit the same
  // bin in one instruction are not what the pass waits for.
  constexpr int kIpUnroll = 4;
  auto load_keys4 = [&](int i4, unsigned int (&key)[4]) -> bool {  // keys of positions 4*i4 .. 4*i4+3
    const bool act = i4 < n4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (act) {
      v = __ldg(reinterpret_cast<const float4*>(A) + i4);
      const int left = n_loc - 4 * i4;
      if (left < 4) v.w = 0.f;
      if (left < 3) v.z = 0.f;
      if (left < 2) v.y = 0.f;
    }
    key[0] = __float_as_uint(v.x + 0.f);  // -0.0 reads as +0.0
    key[1] = __float_as_uint(v.y + 0.f);
    key[2] = __float_as_uint(v.z + 0.f);
    key[3] = __float_as_uint(v.w + 0.f);
    return act;
  };
  const int n_pos4 = n4 * 4;                       // slice length rounded up to whole float4s
  const int n_chunks = (n_pos4 + kChunk - 1) / kChunk;
  // selection at chunk granularity: the searched row (one score per chunk) is built after the
  // aggregation, and the search and the compaction walk n_srch entries instead of n_loc
  const bool chunked = kVariant && P.chunk > 1;
  const int n_srch = chunked ? (n_loc + P.chunk - 1) / P.chunk : n_loc;
  // Alg. 2 as printed selects per speculated query and unions the sets: then everything up to
  // the threshold runs once per query over the row summed over heads only, and the kept
  // positions are collected in a bit mask of the slice.
  const int n_steps = (kVariant && P.per_step) ? P.gamma : 1;
  unsigned int theta_key = 0u;  // keep everything with key >= theta_key
  double total = 0.0, target = 0.0, m_gt = 0.0, m_ge = 0.0;
  bool invalid = false;
  if (tid == 0) sh.n_invalid = 0;
  bool short_cut = false;  // the threshold was found among the gathered keys of the level-1 bin
  bool tie_done = false;   // (rows read in place) the threshold bin held one distinct value: the threshold
  // (in place) the kept positions as ballot words, four per 128 positions, in the upper half of
  // the scan array: by the time they are written the level-1 scan is over, the later levels use
  // the lower half only, and no peer reads this array after the level-1 gather
  unsigned int* const keep_words = reinterpret_cast<unsigned int*>(r_mass + kL23Bins);
  for (int step = 0; step < n_steps; ++step) {
  // contributing rows in the order that defines the aggregated value
  if (tid == 0) {
    int n = 0;
    if (kInPlace) {
      n = 1;
    } else {
      for (int h = 0; h < P.H; ++h) {
        if (P.has_groups && P.head_group[h] != g) continue;
        if (kVariant && P.per_step) {
          row_off[n++] = static_cast<long long>(h * P.gamma + step) * P.L_stride;
        } else {
          for (int s = 0; s < P.gamma; ++s) row_off[n++] = static_cast<long long>(h * P.gamma + s) * P.L_stride;
        }
      }
    }
    sh.n_rows = n;
    sh.n_cand = 0;
    sh.bin_lo = kL1Bins;
    sh.bin_hi = -1;
  }
  for (int i = tid; i < kL1Bins; i += kThreads) sh.h_hi[i] = sh.h_lo[i] = 0u;
  __syncthreads();
  // two-launch form: this kernel was allowed to start while the aggregation still ran
  if (kInPlace && P.agg != nullptr) pdl_wait();
  const int R = sh.n_rows;
  float vmax = 0.f;  // largest aggregated value of this thread's positions (literal bisection)

  // ---- 1+2: aggregate the slice and build the level-1 histogram ------------------------------
  bool bad = false;
  if (in_place) {
    // single contributing row: one pass over the slice for validity and the level-1 histogram.
    // The pass is bound by instruction issue, so whole iterations (every float4 of the CTA inside
    // the slice and complete: all but the last one or two) run a lean body: validity through a
    // running maximum of the bit patterns (a negative, NaN or infinite value is a pattern above
    // 0x7f7fffff), no bounds tests, and the test "does the whole warp hit one bin" (ties) once
    // per 16 values of a thread instead of once per 4.
    int ip_main = 0;
    if (!kVariant) {
      unsigned int kbits = 0u;
      for (; ip_main < n4_main; ip_main += kIpUnroll * kThreads) {
        float4 v[kIpUnroll];
#pragma unroll
        for (int uu = 0; uu < kIpUnroll; ++uu)
          v[uu] = __ldg(reinterpret_cast<const float4*>(A) + ip_main + uu * kThreads + tid);
        unsigned int k[kIpUnroll * 4];
        unsigned int k_or = 0u, k_and = 0xffffffffu;
#pragma unroll
        for (int uu = 0; uu < kIpUnroll; ++uu) {
          k[4 * uu + 0] = __float_as_uint(v[uu].x + 0.f);  // -0.0 reads as +0.0
          k[4 * uu + 1] = __float_as_uint(v[uu].y + 0.f);
          k[4 * uu + 2] = __float_as_uint(v[uu].z + 0.f);
          k[4 * uu + 3] = __float_as_uint(v[uu].w + 0.f);
        }
#pragma unroll
        for (int j = 0; j < kIpUnroll * 4; ++j) {
          kbits = max(kbits, k[j]);
          k_or |= k[j];
          k_and &= k[j];
        }
        // all 16 values of this thread in one bin, and the same bin in every lane: one reduction
        // per word for the warp (zeros can only share bin 0, where they add nothing)
        const unsigned int my_bin = k[0] >> 20;
        const bool mine_same = ((k_or ^ k_and) >> 20) == 0u && !(k_or >> 31);  // (a set sign bit: invalid input)
        const unsigned int bin0 = __shfl_sync(kFull, my_bin, 0);  // (every lane takes part: not inside the &&)
        if (__all_sync(kFull, mine_same && my_bin == bin0)) {
          unsigned int lo = 0u, hi = 0u;
#pragma unroll
          for (int j = 0; j < kIpUnroll * 4; ++j) {
            const unsigned int m = mantissa_of(k[j]);
            lo += m & 0xffffu;
            hi += m >> 16;
          }
          lo = __reduce_add_sync(kFull, lo);
          hi = __reduce_add_sync(kFull, hi);
          if (lane == 0) hist_bump(h1, static_cast<int>(my_bin), lo, hi);
        } else {
#pragma unroll
          for (int j = 0; j < kIpUnroll * 4; ++j) {
            const unsigned int m = mantissa_of(k[j]);
            if (k[j] != 0u && !(k[j] >> 31)) hist_bump(h1, static_cast<int>(k[j] >> 20), m & 0xffffu, m >> 16);
          }
        }
      }
      bad |= kbits > 0x7f7fffffu;
    }
    // the rest of the slice (and everything, for the variants): bounds and validity per value
    for (int base = ip_main; base < n4; base += kIpUnroll * kThreads) {
      unsigned int key[kIpUnroll][4];
      bool act[kIpUnroll];
#pragma unroll
      for (int uu = 0; uu < kIpUnroll; ++uu) act[uu] = load_keys4(base + uu * kThreads + tid, key[uu]);
#pragma unroll
      for (int uu = 0; uu < kIpUnroll; ++uu) {
        const int i4 = base + uu * kThreads + tid;
        bool take[4];
        int bin[4];
        unsigned int mant[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned int k = key[uu][e];
          // negative, NaN or infinite: sign bit set, or an all-ones exponent
          bad |= act[uu] && k > 0x7f7fffffu;
          if (kVariant && !chunked) vmax = fmaxf(vmax, __uint_as_float(k));
          take[e] = act[uu] && (4 * i4 + e < n_loc) && k != 0u && !(k >> 31) && !chunked;
          bin[e] = static_cast<int>(k >> 20);
          mant[e] = mantissa_of(k);
        }
        hist_add4(h1, take, bin, mant);
      }
    }
  } else
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
        const float* src = src0 + row_off[ir] + ic * kChunk;
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
    int slot_c = 0;
    for (int c = 0; c < n_chunks; ++c) {
      const int len4 = min(kChunk, n_pos4 - c * kChunk) >> 2;
      // positions of this thread's two float4s that lie beyond the slice (last float4 only)
      int cut[2];
#pragma unroll
      for (int k = 0; k < 2; ++k) cut[k] = n_loc - (c * kChunk + 4 * (tid + k * kThreads));
      for (int r = 0; r < R; ++r) {
        issue();
        asm volatile("cp.async.wait_group %0;" ::"n"(kDepth - 1) : "memory");
        const float4* piece = reinterpret_cast<const float4*>(ring + slot_c * kChunk);
        slot_c = (slot_c + 1) & (kDepth - 1);
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int i4 = tid + k * kThreads;
          if (i4 < len4) {
            float4 x = piece[i4];
            if (cut[k] < 4) {  // values beyond kv_len are not inputs
              x.w = 0.f;
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
        if (kVariant && act && !chunked) vmax = fmaxf(vmax, fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)));
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned int key = __float_as_uint(vals[e]);
          // zeros carry no mass and can never be the threshold of a row with positive total
          const bool take = act && (pos + e < n_loc) && key != 0u && !(key >> 31) && !chunked;
          hist_add(h1, take, static_cast<int>(key >> 20), mantissa_of(key));
        }
        acc[k] = mn[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  }
  if (chunked) {
    // Selection at chunk granularity: entry j of the searched row is the binary32 sum of the
    // chunk's aggregated values in ascending order (the last chunk of the list is cut at L).
    // The scores replace the head of the slice: a round reads 256 chunks, then writes 256
    // entries that no later round reads.
    __syncthreads();  // the aggregated slice is complete
    for (int base = 0; base < n_srch; base += kThreads) {
      const int j = base + tid;
      const bool act = j < n_srch;
      float acc = 0.f;
      if (act) {
        const int p0 = j * P.chunk;
        for (int e = 0; e < P.chunk; e += 4) {
          const float4 v = *reinterpret_cast<const float4*>(a + p0 + e);
          const int left = n_loc - (p0 + e);
          if (left > 0) acc = acc + v.x;
          if (left > 1) acc = acc + v.y;
          if (left > 2) acc = acc + v.z;
          if (left > 3) acc = acc + v.w;
        }
      }
      __syncthreads();
      if (act) {
        a[j] = acc;
        bad |= !(acc <= FLT_MAX);
        vmax = fmaxf(vmax, acc);
      }
      const unsigned int key = __float_as_uint(acc);
      hist_add(h1, act && key != 0u && !(key >> 31), static_cast<int>(key >> 20), mantissa_of(key));
    }
  }
  if (bad) atomicAdd(&sh.n_invalid, 1);
  if (kVariant) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) vmax = fmaxf(vmax, __shfl_xor_sync(kFull, vmax, o));
    if (lane == 0) sh.warp_max[warp] = vmax;
  }
  __syncthreads();
  if (kVariant && tid == 0) {
    float m = 0.f;
    for (int w = 0; w < kWarps; ++w) m = fmaxf(m, sh.warp_max[w]);
    sh.cta_max = m;
  }
  // the ring is idle from here on: zero this CTA's level-2 and level-3 histograms
  for (int i = tid; i < 2 * 2 * kL23Bins; i += kThreads) lvl_base[i] = 0u;
  {
    // first and last non-empty bin of the level-1 histogram (complete since the barrier above):
    // rows of attention probabilities fill a few hundred of the 2048 bins, and the cluster
    // reduction and the scan below then touch only those
    int bmin = kL1Bins, bmax = -1;
    for (int bin = tid; bin < kL1Bins; bin += kThreads) {
      if ((sh.h_lo[bin] | sh.h_hi[bin]) != 0u) {
        bmin = min(bmin, bin);
        bmax = max(bmax, bin);
      }
    }
    bmin = __reduce_min_sync(kFull, bmin);
    bmax = __reduce_max_sync(kFull, bmax);
    if (lane == 0 && bmax >= 0) {
      atomicMin(&sh.bin_lo, bmin);
      atomicMax(&sh.bin_hi, bmax);
    }
  }
  __syncthreads();

  // ---- 3: threshold search --------------------------------------------------------------------
  csync();  // every CTA's level-1 histogram and invalid count are complete
  int n_bad = 0, glo = kL1Bins, ghi = -1;
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    if (r < cs) {
      n_bad += *cluster.map_shared_rank(&sh.n_invalid, r);
      glo = min(glo, *cluster.map_shared_rank(&sh.bin_lo, r));
      ghi = max(ghi, *cluster.map_shared_rank(&sh.bin_hi, r));
    }
  }
  // whole scan groups; an empty histogram gives an empty range
  glo = (ghi < 0) ? 0 : (glo & ~(kGroup - 1));
  ghi = (ghi < 0) ? 0 : ((ghi | (kGroup - 1)) + 1);
  // one or two CTAs: every CTA sums the bins over the ranks itself (one cluster barrier and the
  // gather less).  Larger clusters: each CTA reduces its own share of the bins and all gather the
  // result (all-to-all reads of every histogram by eight CTAs cost more than that barrier).
  const bool narrow = cs <= 2;

  theta_key = 0u;
  invalid = n_bad != 0;  // the count only grows from step to step: the last one decides
  bool searching = !invalid;
  if (searching && narrow) {
    for (int bin = glo + tid; bin < ghi; bin += kThreads) {
      unsigned long long mh = 0, ml = 0;
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        if (r < cs) {
          mh += *cluster.map_shared_rank(&sh.h_hi[bin], r);
          ml += *cluster.map_shared_rank(&sh.h_lo[bin], r);
        }
      }
      r_mass[bin] = static_cast<double>((mh << 16) + ml) * pow2_double(max(bin >> 3, 1) - 150);
    }
  } else if (searching) {
    // level 1: every CTA reduces its own range of bins over the cluster, then all gather
    const int per_bins = kL1Bins / cs;
    const int blo = max(rank * per_bins, glo), bhi = min((rank + 1) * per_bins, ghi);
    for (int bin = blo + tid; bin < bhi; bin += kThreads) {
      unsigned long long mh = 0, ml = 0;
      for (int r = 0; r < cs; ++r) {
        mh += *cluster.map_shared_rank(&sh.h_hi[bin], r);
        ml += *cluster.map_shared_rank(&sh.h_lo[bin], r);
      }
      r_mass[bin] = static_cast<double>((mh << 16) + ml) * pow2_double(max(bin >> 3, 1) - 150);
    }
  }
  if (!narrow) csync();  // every owner's range is reduced
  if (searching) {
    if (!narrow) {
      const int per_bins = kL1Bins / cs;
      for (int bin = glo + tid; bin < ghi; bin += kThreads) {
        const int owner = bin / per_bins;
        if (owner != rank) r_mass[bin] = *cluster.map_shared_rank(&r_mass[bin], owner);
      }
    }
  }
  // (rows read in place) the ballot words of the kept positions overlay the upper half of this
  // array from the candidate pass on: no CTA may get there while a peer still gathers from it
  if (kInPlace && !narrow) csync();
  if (searching) {
    __syncthreads();
    scan_bins(sh, r_mass, kL1Bins, 0.0, 0.0, true, P.p, glo / kGroup, ghi / kGroup);
    total = sh.total;
    target = static_cast<double>(P.p) * total;
    m_ge = total;
    searching = (target > 0.0) && !P.keep_all;  // else: p >= 1 or an all-zero row -> keep all
  }
  // Levels 2 and 3 refine inside the found bin.  The cluster syncs are executed by every
  // CTA whatever it decided (the decisions are identical across the cluster anyway).
  unsigned int prefix = searching ? static_cast<unsigned int>(sh.found_bin) : 0u;
  const int e1 = max(static_cast<int>(prefix >> 3), 1) - 150;
  double carry_m = searching ? sh.mass_above : 0.0;
  short_cut = false;
  // Short cut: the threshold bin of level 1 usually holds few values (tens to hundreds for
  // attention rows).  Its mantissa sum S bounds their number (a normal mantissa is >= 2^23); when
  // at most kCandCap fit, every CTA collects its keys of that bin, fetches everybody's, and
  // finds the threshold among them directly -- the sums of their mantissas are exact integers,
  // so every CTA decides alike -- instead of two more rounds of histogram, cluster reduction
  // and scan (~6 us each, all latency).
  if (searching && (prefix >> 3) >= 1u) {
    const unsigned long long S = static_cast<unsigned long long>(r_mass[prefix] * pow2_double(-e1));
    short_cut = (S >> 23) <= static_cast<unsigned long long>(kCandCap);
  }
  // every thread has read the bin's mass before a faster warp's ballot words can land on it
  if (kInPlace) __syncthreads();
  // What the candidates are: the keys whose bits above `csh` equal `cpre` -- the level-1 bin
  // (11 bits), or, after the merged pass below, a level-2 bin inside it (21 bits).
  int csh = 20, lvl0 = 0;
  unsigned int cpre = prefix;
  tie_done = false;
  bool level2_done = false;  // the merged pass ran but its bin is too full for the short cut
  const double m_ge_l1 = searching ? sh.mass_ge : 0.0;
  if (kInPlace && !kVariant && searching && !short_cut) {
    // Rows read in place whose threshold bin is well filled (flat or tie-heavy rows).  Every pass
    // over such a row costs as much as the level-1 pass, so the second one does three things at
    // once: it notes the positions inside or above the threshold bin as ballot words, builds the
    // level-2 histogram of the bin, and tracks the smallest and largest key inside the bin.  If
    // those are equal (ties) the search is over and the ballot words are the kept set; otherwise
    // the level-2 bin found is normally sparse enough for the short cut, whose candidate pass
    // then is the third and last pass over the row (five before: two more histogram levels, a
    // count pass and the write pass's own read).
    unsigned int* const lb2 = lvl_base;                                  // level-2 histogram
    const Hist hr = {lb2, lb2 + kL23Bins};
    unsigned int kmin = 0xffffffffu, kmax = 0u;
    // whole iterations: no bounds tests; the histogram is only touched for float4s in which some
    // lane holds a value of the bin
    int mp_main = 0;
    for (; mp_main < n4_main; mp_main += kIpUnroll * kThreads) {
      float4 v[kIpUnroll];
#pragma unroll
      for (int uu = 0; uu < kIpUnroll; ++uu)
        v[uu] = __ldg(reinterpret_cast<const float4*>(A) + mp_main + uu * kThreads + tid);
#pragma unroll
      for (int uu = 0; uu < kIpUnroll; ++uu) {
        const unsigned int k[4] = {__float_as_uint(v[uu].x + 0.f), __float_as_uint(v[uu].y + 0.f),
                                   __float_as_uint(v[uu].z + 0.f), __float_as_uint(v[uu].w + 0.f)};
        bool take[4];
        bool all_in = true;
        unsigned int mine = 0u;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned int top = k[e] >> 20;
          take[e] = top == prefix;
          all_in &= take[e];
          const unsigned int m = __ballot_sync(kFull, top >= prefix);
          if (lane == e) mine = m;
        }
        // Every value of the warp's 128 inside the bin (constant or near-constant rows): the tie
        // test and the warp-wide reduction of hist_add4.  Otherwise the bin holds a few per cent
        // of the values and each of them updates the histogram on its own.
        if (__all_sync(kFull, all_in)) {
          int bin[4];
          unsigned int mant[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            bin[e] = static_cast<int>((k[e] >> 10) & 1023u);
            mant[e] = mantissa_of(k[e]);
            kmin = min(kmin, k[e]);
            kmax = max(kmax, k[e]);
          }
          hist_add4(hr, take, bin, mant);
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            if (take[e]) {
              const unsigned int m = mantissa_of(k[e]);
              hist_bump(hr, static_cast<int>((k[e] >> 10) & 1023u), m & 0xffffu, m >> 16);
              kmin = min(kmin, k[e]);
              kmax = max(kmax, k[e]);
            }
          }
        }
        if (lane < 4) keep_words[((mp_main + uu * kThreads + (tid & ~31)) >> 5) * 4 + lane] = mine;
      }
    }
    for (int base = mp_main; base < n4; base += kIpUnroll * kThreads) {
      unsigned int key[kIpUnroll][4];
      bool act[kIpUnroll];
#pragma unroll
      for (int uu = 0; uu < kIpUnroll; ++uu) act[uu] = load_keys4(base + uu * kThreads + tid, key[uu]);
#pragma unroll
      for (int uu = 0; uu < kIpUnroll; ++uu) {
        const int i4 = base + uu * kThreads + tid;
        unsigned int mine = 0u;
        bool take[4];
        int bin[4];
        unsigned int mant[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned int k = key[uu][e];
          const bool in_row = act[uu] && (4 * i4 + e < n_loc);
          const bool inb = in_row && (k >> 20) == prefix;
          take[e] = inb;
          bin[e] = static_cast<int>((k >> 10) & 1023u);
          mant[e] = mantissa_of(k);
          kmin = inb ? min(kmin, k) : kmin;
          kmax = inb ? max(kmax, k) : kmax;
          // in the bin or above it: exactly the kept set if the bin turns out to hold one value
          const unsigned int m = __ballot_sync(kFull, in_row && (k >> 20) >= prefix);
          if (lane == e) mine = m;
        }
        hist_add4(hr, take, bin, mant);
        const int g4 = base + uu * kThreads + (tid & ~31);  // first float4 of this warp's 32
        if (lane < 4 && g4 < n4) keep_words[(g4 >> 5) * 4 + lane] = mine;
      }
    }
    kmin = __reduce_min_sync(kFull, kmin);
    kmax = __reduce_max_sync(kFull, kmax);
    if (lane == 0) {
      sh.red_key[warp] = kmin;
      sh.red_key[kWarps + warp] = kmax;
    }
    __syncthreads();
    if (tid == 0) {
      unsigned int a0 = 0xffffffffu, a1 = 0u;
      for (int w = 0; w < kWarps; ++w) {
        a0 = min(a0, sh.red_key[w]);
        a1 = max(a1, sh.red_key[kWarps + w]);
      }
      sh.bin_kmin = a0;
      sh.bin_kmax = a1;
    }
    csync();  // every CTA's level-2 histogram and key range are complete
    kmin = 0xffffffffu;
    kmax = 0u;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      if (r < cs) {
        kmin = min(kmin, *cluster.map_shared_rank(&sh.bin_kmin, r));
        kmax = max(kmax, *cluster.map_shared_rank(&sh.bin_kmax, r));
      }
    }
    if (kmin == kmax) {
      // one distinct value in the bin: it is the threshold, and all its positions are kept
      theta_key = kmin;
      m_gt = carry_m;
      m_ge = m_ge_l1;
      tie_done = true;
    } else {
      const double scale = pow2_double(e1);
      for (int bin = tid; bin < kL23Bins; bin += kThreads) {
        unsigned long long ml = 0, mh = 0;
        for (int r = 0; r < cs; ++r) {
          const unsigned int* src = cluster.map_shared_rank(lb2, r);
          ml += src[bin];
          mh += src[kL23Bins + bin];
        }
        r_mass[bin] = static_cast<double>((mh << 16) + ml) * scale;
      }
      __syncthreads();
      scan_bins(sh, r_mass, kL23Bins, carry_m, target, false, P.p);
      const unsigned long long S2 =
          static_cast<unsigned long long>(r_mass[sh.found_bin] * pow2_double(-e1));
      prefix = (prefix << 10) | static_cast<unsigned int>(sh.found_bin);
      carry_m = sh.mass_above;
      level2_done = true;
      if ((S2 >> 23) <= static_cast<unsigned long long>(kCandCap)) {
        short_cut = true;
        csh = 10;
        lvl0 = 1;
        cpre = prefix;
      }
      __syncthreads();  // everybody has read r_mass / the scan results before they are reused
    }
  }
  if (short_cut) {
    if (in_place) {
      // whole iterations: no bounds tests, and the candidate list is only touched for float4s in
      // which some lane holds a candidate (a few hundred per row)
      int cp_main = 0;
      for (; cp_main < n4_main; cp_main += kIpUnroll * kThreads) {
        float4 v[kIpUnroll];
#pragma unroll
        for (int uu = 0; uu < kIpUnroll; ++uu)
          v[uu] = __ldg(reinterpret_cast<const float4*>(A) + cp_main + uu * kThreads + tid);
#pragma unroll
        for (int uu = 0; uu < kIpUnroll; ++uu) {
          const int i4 = cp_main + uu * kThreads + tid;
          const unsigned int k[4] = {__float_as_uint(v[uu].x + 0.f), __float_as_uint(v[uu].y + 0.f),
                                     __float_as_uint(v[uu].z + 0.f), __float_as_uint(v[uu].w + 0.f)};
          bool is_cand[4];
          bool any_cand = false;
          unsigned int mine = 0u;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const unsigned int top = k[e] >> csh;
            is_cand[e] = top == cpre;
            any_cand |= is_cand[e];
            const unsigned int m = __ballot_sync(kFull, top > cpre);
            if (lane == e) mine = m;
          }
          if (__any_sync(kFull, any_cand)) {
#pragma unroll
            for (int e = 0; e < 4; ++e) cand_add(sh, is_cand[e], k[e], 4 * i4 + e);
          }
          if (lane < 4) keep_words[((cp_main + uu * kThreads + (tid & ~31)) >> 5) * 4 + lane] = mine;
        }
      }
        for (int base = cp_main; base < n4; base += kIpUnroll * kThreads) {
          unsigned int key[kIpUnroll][4];
        bool act[kIpUnroll];
#pragma unroll
        for (int uu = 0; uu < kIpUnroll; ++uu) act[uu] = load_keys4(base + uu * kThreads + tid, key[uu]);
#pragma unroll
        for (int uu = 0; uu < kIpUnroll; ++uu) {
          const int i4 = base + uu * kThreads + tid;
          // values in a higher bin are kept whatever the threshold turns out to be: their
          // ballot words go where the count pass would put them, and once the threshold is
          // known the candidates that made it are added -- the row is not read a third time
          unsigned int mine = 0u;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const bool in_row = act[uu] && (4 * i4 + e < n_loc);
            cand_add(sh, in_row && (key[uu][e] >> csh) == cpre, key[uu][e], 4 * i4 + e);
            const unsigned int m = __ballot_sync(kFull, in_row && (key[uu][e] >> csh) > cpre);
            if (lane == e) mine = m;
          }
          const int g4 = base + uu * kThreads + (tid & ~31);  // first float4 of this warp's 32
          if (lane < 4 && g4 < n4) keep_words[(g4 >> 5) * 4 + lane] = mine;
        }
      }
    } else {
      for (int base = 0; base < n_srch; base += kThreads) {
        const int i = base + tid;
        const unsigned int key = (i < n_srch) ? key_at(i) : 0u;
        cand_add(sh, i < n_srch && (key >> csh) == cpre, key, i);
      }
    }
    csync();  // every CTA's candidate list is complete
    int cnt_r[8];
    int M = 0;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      cnt_r[r] = (r < cs) ? min(*cluster.map_shared_rank(&sh.n_cand, r), kCandCap) : 0;
      M += cnt_r[r];
    }
    M = min(M, kCandCap);  // (the bound on S guarantees it)
    unsigned int* const all = sh.all_keys;
    int off = 0;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      if (r < cs) {
        const unsigned int* src = cluster.map_shared_rank(sh.cand, r);
        for (int i = tid; i < cnt_r[r] && off + i < kCandCap; i += kThreads) all[off + i] = src[i];
        off += cnt_r[r];
      }
    }
    __syncthreads();
    // More keys: levels 2 and 3 over the gathered keys instead of over the row -- the same exact
    // mantissa sums per bin and the same scan as the cluster-wide levels below, but on at most
    // kCandCap values that every CTA holds itself: no pass over the row, no cluster reduction.
    // (The direct search costs O(M^2): ~6 us at M ~ 400, against ~2 us for the two local levels;
    // below ~128 keys it is the faster of the two.)
    const double scale = pow2_double(e1);
    if (M <= kDirectMax) {
      // few keys: for each one the exact sum of the mantissas of the keys >= it; the highest key
      // whose suffix (itself, its ties and everything above) reaches the target is the threshold
      unsigned int best = 0u, lowest = 0xffffffffu;
      for (int i = tid; i < M; i += kThreads) {
        const unsigned int ki = all[i];
        unsigned long long s_ge = 0ull;
        for (int j = 0; j < M; ++j) {
          const unsigned int kj = all[j];
          s_ge += (kj >= ki) ? mantissa_of(kj) : 0u;
        }
        if (carry_m + static_cast<double>(s_ge) * scale >= target) best = max(best, ki);
        lowest = min(lowest, ki);
      }
      best = __reduce_max_sync(kFull, best);
      lowest = __reduce_min_sync(kFull, lowest);
      if (lane == 0) {
        sh.red_key[warp] = best;
        sh.red_key[kWarps + warp] = lowest;
      }
      __syncthreads();
      best = 0u;
      lowest = 0xffffffffu;
      for (int w = 0; w < kWarps; ++w) {
        best = max(best, sh.red_key[w]);
        lowest = min(lowest, sh.red_key[kWarps + w]);
      }
      // (no key reaches it only through rounding between two summation orders: keep the bin)
      const unsigned int theta = (best != 0u) ? best : lowest;
      unsigned long long s_ge = 0ull, s_gt = 0ull;
      for (int j = tid; j < M; j += kThreads) {
        const unsigned int kj = all[j];
        s_ge += (kj >= theta) ? mantissa_of(kj) : 0u;
        s_gt += (kj > theta) ? mantissa_of(kj) : 0u;
      }
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) {
        s_ge += __shfl_xor_sync(kFull, s_ge, o);
        s_gt += __shfl_xor_sync(kFull, s_gt, o);
      }
      if (lane == 0) {
        sh.red_sum[warp] = s_ge;
        sh.red_sum[kWarps + warp] = s_gt;
      }
      __syncthreads();
      s_ge = s_gt = 0ull;
      for (int w = 0; w < kWarps; ++w) {
        s_ge += sh.red_sum[w];
        s_gt += sh.red_sum[kWarps + w];
      }
      theta_key = theta;
      m_gt = carry_m + static_cast<double>(s_gt) * scale;
      m_ge = carry_m + static_cast<double>(s_ge) * scale;
    } else {
    unsigned int pre = cpre;
    double carry = carry_m;
#pragma unroll 1
    for (int level = lvl0; level < 2; ++level) {
      const int shift = (level == 0) ? 10 : 0;
      unsigned int* lb = lvl_base + level * 2 * kL23Bins;  // zeroed above; the cluster does not use it on this path
      const Hist hr = {lb, lb + kL23Bins};
      for (int i = tid; i < M; i += kThreads) {
        const unsigned int k = all[i];
        if ((k >> (shift + 10)) == pre) {
          const unsigned int mant = mantissa_of(k);
          hist_bump(hr, static_cast<int>((k >> shift) & 1023u), mant & 0xffffu, mant >> 16);
        }
      }
      __syncthreads();
      for (int bin = tid; bin < kL23Bins; bin += kThreads)
        r_mass[bin] = static_cast<double>((static_cast<unsigned long long>(lb[kL23Bins + bin]) << 16) + lb[bin]) * scale;
      __syncthreads();
      scan_bins(sh, r_mass, kL23Bins, carry, target, false, P.p);
      pre = (pre << 10) | static_cast<unsigned int>(sh.found_bin);
      carry = sh.mass_above;
    }
    theta_key = pre;
    m_gt = sh.mass_above;
    m_ge = sh.mass_ge;
    }
    if (in_place && !kVariant) {
      // this CTA's candidates that reach the threshold join the positions recorded above
      const int n_own = min(sh.n_cand, kCandCap);
      __syncthreads();  // the ballot words of the candidate pass are complete
      for (int i = tid; i < n_own; i += kThreads) {
        if (sh.cand[i] >= theta_key) {
          const int pos = sh.cand_pos[i];
          atomicOr(&keep_words[(pos >> 7) * 4 + (pos & 3)], 1u << ((pos >> 2) & 31));
        }
      }
      __syncthreads();
    }
  } else if (!tie_done) {
  for (int level = level2_done ? 1 : 0; level < 2; ++level) {
    const int shift = (level == 0) ? 10 : 0;
    unsigned int* lb = lvl_base + level * 2 * kL23Bins;
    if (searching) {
      // only the elements inside the threshold bin take part
      const Hist hr = {lb, lb + kL23Bins};
      if (in_place) {
            for (int base = 0; base < n4; base += kIpUnroll * kThreads) {
              unsigned int key[kIpUnroll][4];
          bool act[kIpUnroll];
#pragma unroll
          for (int uu = 0; uu < kIpUnroll; ++uu) act[uu] = load_keys4(base + uu * kThreads + tid, key[uu]);
#pragma unroll
          for (int uu = 0; uu < kIpUnroll; ++uu) {
            const int i4 = base + uu * kThreads + tid;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const bool take = act[uu] && (4 * i4 + e < n_loc) && (key[uu][e] >> (shift + 10)) == prefix;
              hist_add(hr, take, static_cast<int>((key[uu][e] >> shift) & 1023u), mantissa_of(key[uu][e]));
            }
          }
        }
      } else
      for (int base = 0; base < n_srch; base += kThreads) {
        const int i = base + tid;
        unsigned int key = 0u;
        bool take = false;
        if (i < n_srch) {
          key = key_at(i);
          take = (key >> (shift + 10)) == prefix;
        }
        hist_add(hr, take, static_cast<int>((key >> shift) & 1023u), mantissa_of(key));
      }
    }
    csync();  // every CTA's histogram of this level is complete
    if (searching) {
      const double scale = pow2_double(e1);
      for (int bin = tid; bin < kL23Bins; bin += kThreads) {
        unsigned long long ml = 0, mh = 0;
        for (int r = 0; r < cs; ++r) {
          const unsigned int* src = cluster.map_shared_rank(lb, r);
          ml += src[bin];
          mh += src[kL23Bins + bin];
        }
        r_mass[bin] = static_cast<double>((mh << 16) + ml) * scale;
      }
      __syncthreads();
      scan_bins(sh, r_mass, kL23Bins, carry_m, target, false, P.p);
      prefix = (prefix << 10) | static_cast<unsigned int>(sh.found_bin);
      carry_m = sh.mass_above;
    }
  }
  }
  if (searching && !short_cut && !tie_done) {
    theta_key = prefix;
    m_gt = sh.mass_above;
    m_ge = sh.mass_ge;
  }
  if (kVariant) {
    if (searching && P.bisect_iters > 0) {
      // Alg. 2's loop, literally: theta_high = max, theta_low = 0, n midpoints in binary32.  The
      // mass of {a >= theta} does not grow with theta, so "mass(theta_mid) < target" holds
      // exactly when theta_mid lies above the exact threshold found above: the midpoints are
      // those of the printed loop without another pass over the row.
      float th_hi = 0.f, th_lo = 0.f, th_mid = 0.f;
      for (int r = 0; r < cs; ++r) th_hi = fmaxf(th_hi, *cluster.map_shared_rank(&sh.cta_max, r));
      for (int it = 0; it < P.bisect_iters; ++it) {
        th_mid = __fmul_rn(__fadd_rn(th_hi, th_lo), 0.5f);
        if (__float_as_uint(th_mid) > theta_key) th_hi = th_mid; else th_lo = th_mid;
      }
      theta_key = __float_as_uint(th_mid);
    }
    if (P.per_step) {
      // collect this query's set in the mask: a warp owns whole 32-position words
      unsigned int* mask = reinterpret_cast<unsigned int*>(ring + kRingFloats);
      const int chunk_m = (((n_srch + kWarps - 1) / kWarps) + 31) & ~31;
      const int m_lo = min(n_srch, warp * chunk_m), m_hi = min(n_srch, m_lo + chunk_m);
      for (int i0 = m_lo; i0 < m_hi; i0 += 32) {
        const int i = i0 + lane;
        const bool keep = !invalid && i < m_hi && key_at(i) >= theta_key;
        const unsigned int m = __ballot_sync(kFull, keep);
        if (lane == 0) mask[i0 >> 5] = (step == 0) ? m : (mask[i0 >> 5] | m);
      }
      // the next query's row overwrites the slice and the staging ring, which peers may still
      // be reading (their scans of this CTA's last histogram)
      csync();
    }
  }
  }  // for step

  // ---- 4: ordered compaction --------------------------------------------------------------------
  // per-warp contiguous ranges of the searched entries, 32 per step; an entry stands for one
  // position, or for the positions of one chunk (all `chunk` of them, except the last chunk of
  // the list, which nothing follows)
  const int wchunk = (((n_srch + kWarps - 1) / kWarps) + 31) & ~31;
  const int w_lo = min(n_srch, warp * wchunk);
  const int w_hi = min(n_srch, w_lo + wchunk);
  const unsigned int* const kept_mask = reinterpret_cast<const unsigned int*>(ring + kRingFloats);
  auto kept = [&](int i) -> bool {
    if (kVariant && P.per_step) return (kept_mask[i >> 5] >> (i & 31)) & 1u;
    return key_at(i) >= theta_key;
  };
  auto n_pos = [&](int i) -> int { return chunked ? min(P.chunk, n_loc - i * P.chunk) : 1; };
  // a row read in place: per-warp ranges of whole float4s, four loads per lane in flight
  const int wchunk4 = (((n4 + kWarps - 1) / kWarps) + 31) & ~31;
  const int w4_lo = min(n4, warp * wchunk4);
  const int w4_hi = min(n4, w4_lo + wchunk4);
  int wc = 0;
  if (!invalid && in_place && !kVariant && (short_cut || tie_done)) {
    // the kept positions are already in the ballot words: count this warp's
    // (a warp whose range is empty has w4_lo == w4_hi == n4, not a multiple of 32)
    if (w4_lo < w4_hi)
      for (int w = (w4_lo >> 5) * 4 + lane; w < ((w4_hi + 31) >> 5) * 4; w += 32) wc += __popc(keep_words[w]);
    wc = __reduce_add_sync(kFull, wc);
  } else if (!invalid && in_place) {
    for (int i0 = w4_lo; i0 < w4_hi; i0 += 32 * kIpUnroll) {
      unsigned int key[kIpUnroll][4];
      bool act[kIpUnroll];
#pragma unroll
      for (int uu = 0; uu < kIpUnroll; ++uu) {
        const int i4 = i0 + uu * 32 + lane;
        act[uu] = load_keys4(i4 < w4_hi ? i4 : n4, key[uu]);
      }
#pragma unroll
      for (int uu = 0; uu < kIpUnroll; ++uu) {
        // 128 consecutive positions, four per lane: one ballot word per position-in-float4.
        // The words are kept (lane e stores word e), so the write pass below never reads the
        // row again.
        const int i4 = i0 + uu * 32 + lane;
        unsigned int mine = 0u;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned int m = __ballot_sync(kFull, act[uu] && 4 * i4 + e < n_loc && key[uu][e] >= theta_key);
          wc += __popc(m);
          if (lane == e) mine = m;
        }
        if (lane < 4 && i0 + uu * 32 < w4_hi) keep_words[((i0 + uu * 32) >> 5) * 4 + lane] = mine;
      }
    }
  } else if (!invalid) {
    for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
      const int i = i0 + lane;
      const bool keep = i < w_hi && kept(i);
      if (chunked) wc += __reduce_add_sync(kFull, keep ? n_pos(i) : 0);
      else wc += __popc(__ballot_sync(kFull, keep));
    }
  }
  if (lane == 0) sh.warp_cnt[warp] = wc;
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
  csync();  // local_kept of every CTA is visible
  long long offset = 0, count = 0;
  for (int r = 0; r < cs; ++r) {
    const int c = *cluster.map_shared_rank(&sh.local_kept, r);
    if (r < rank) offset += c;
    count += c;
  }
  if (!invalid && in_place) {
    int* out = P.idx + out_list * P.idx_stride;
    long long pos = offset + sh.warp_cnt[warp];
    const unsigned int lt = (1u << lane) - 1u;
    // (the candidate arrays are idle by now -- every peer is past its gather -- and hold the
    // eight warps' staging lines of 128 positions)
    static_assert(offsetof(Shared, all_keys) - offsetof(Shared, cand) == 2 * kCandCap * sizeof(int) &&
                      3 * kCandCap >= kWarps * 128,
                  "the candidate arrays are contiguous and hold one staging line per warp");
    int* const stage = reinterpret_cast<int*>(sh.cand) + warp * 128;
    __syncwarp();  // this warp's ballot words are complete
    // one group of 128 positions per trip; the next group's ballot words are loaded before this
    // one is worked on, and a group without a kept position (most groups of a peaked row) costs
    // nothing more
    uint4 words = (w4_lo < w4_hi) ? *reinterpret_cast<const uint4*>(keep_words + (w4_lo >> 5) * 4)
                                  : make_uint4(0u, 0u, 0u, 0u);
    for (int g4 = w4_lo; g4 < w4_hi; g4 += 32) {
      const uint4 cur = words;
      if (g4 + 32 < w4_hi) words = *reinterpret_cast<const uint4*>(keep_words + ((g4 + 32) >> 5) * 4);
      if ((cur.x | cur.y | cur.z | cur.w) == 0u) continue;  // (the same words in every lane)
      // 128 consecutive positions, four per lane: ascending order is lane-major
      const int i4 = g4 + lane;
      const unsigned int mw[4] = {cur.x, cur.y, cur.z, cur.w};
      unsigned int before = 0, total_kept = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        before += __popc(mw[e] & lt);
        total_kept += __popc(mw[e]);
      }
      // The kept positions of the 128 go through a per-warp staging line, so that the global
      // stores are whole 128-byte runs (a lane storing its own up to four positions spreads every
      // store instruction over the whole 512-byte range: four partial writes per sector).
      unsigned int at = before;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if ((mw[e] >> lane) & 1u) stage[at++] = lo + 4 * i4 + e;
      }
      __syncwarp();
      for (unsigned int t = lane; t < total_kept; t += 32)
        if (pos + t < P.idx_stride) out[pos + t] = stage[t];
      __syncwarp();
      pos += total_kept;
    }
  } else if (!invalid) {
    int* out = P.idx + out_list * P.idx_stride;
    long long pos = offset + sh.warp_cnt[warp];
    for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
      const int i = i0 + lane;
      const bool keep = i < w_hi && kept(i);
      const unsigned m = __ballot_sync(kFull, keep);
      if (chunked) {
        const int np = keep ? n_pos(i) : 0;
        const long long my = pos + static_cast<long long>(__popc(m & ((1u << lane) - 1u))) * P.chunk;
        for (int e = 0; e < np; ++e)
          if (my + e < P.idx_stride) out[my + e] = lo + i * P.chunk + e;
        pos += __reduce_add_sync(kFull, np);
      } else {
        const long long my = pos + __popc(m & ((1u << lane) - 1u));
        if (keep && my < P.idx_stride) out[my] = lo + i;
        pos += __popc(m);
      }
    }
  }
  if (rank == 0 && tid == 0) {
    int st = SPECATTN_ROW_OK;
    if (invalid) {
      st = SPECATTN_ROW_INVALID_PROB;
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
  csync();  // nobody leaves while its shared memory may still be read remotely
}

// First launch of the two-launch form: a[i] = +0 + the contributing rows in order, for 512
// positions per CTA, so that the number of CTAs streaming the rows from HBM does not depend on
// the number of lists.  The adds are the ones of the cluster kernel (binary32, same order), so
// the bits of a[] are the same.  A negative input, which a sum could hide, poisons its
// position with NaN: the search then reports the list as invalid like the cluster kernel does.
constexpr int kAggThreads = 128;
constexpr int kAggPositions = kAggThreads * 4;
constexpr int kAggUnroll = 16;
__global__ void __launch_bounds__(kAggThreads) aggregate_rows_kernel(const __grid_constant__ SelectParams P,
                                                                  float* __restrict__ out) {
  __shared__ long long row_off[SPECATTN_MAX_ROWS_PER_LIST];
  __shared__ int n_rows;
  const int tid = threadIdx.x;
  const int list = blockIdx.y;
  const int g = list % P.G;
  const int b = (list / P.G) % P.B;
  const int slot = list / (P.G * P.B);
  long long Lll = P.kv_len[b];
  if (Lll < 0) Lll = 0;
  if (Lll > P.L_stride) Lll = P.L_stride;
  const int L = static_cast<int>(Lll);
  const int pos = blockIdx.x * kAggPositions + 4 * tid;
  if (blockIdx.x * kAggPositions >= L) return;
  if (tid == 0) {
    int n = 0;
    for (int h = 0; h < P.H; ++h) {
      if (P.has_groups && P.head_group[h] != g) continue;
      for (int s = 0; s < P.gamma; ++s) row_off[n++] = static_cast<long long>(h * P.gamma + s) * P.L_stride;
    }
    n_rows = n;
  }
  __syncthreads();
  if (pos >= L) return;
  const int R = n_rows;
  const int cut = L - pos;  // positions of this float4 that are inputs
  const float* src = P.probs[slot] + static_cast<long long>(b) * P.H * P.gamma * P.L_stride + pos;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), mn = acc;
  for (int r0 = 0; r0 < R; r0 += kAggUnroll) {
    float4 x[kAggUnroll];
#pragma unroll
    for (int k = 0; k < kAggUnroll; ++k)
      if (r0 + k < R) x[k] = __ldcs(reinterpret_cast<const float4*>(src + row_off[r0 + k]));
#pragma unroll
    for (int k = 0; k < kAggUnroll; ++k) {
      if (r0 + k < R) {
        float4 v = x[k];
        if (cut < 4) {  // values beyond kv_len are not inputs
          v.w = 0.f;
          if (cut < 3) v.z = 0.f;
          if (cut < 2) v.y = 0.f;
        }
        mn.x = fminf(mn.x, v.x);
        mn.y = fminf(mn.y, v.y);
        mn.z = fminf(mn.z, v.z);
        mn.w = fminf(mn.w, v.w);
        acc.x = acc.x + v.x;
        acc.y = acc.y + v.y;
        acc.z = acc.z + v.z;
        acc.w = acc.w + v.w;
      }
    }
  }
  const float nan = __uint_as_float(0x7fc00000u);
  if (mn.x < 0.f) acc.x = nan;
  if (mn.y < 0.f) acc.y = nan;
  if (mn.z < 0.f) acc.z = nan;
  if (mn.w < 0.f) acc.w = nan;
  *reinterpret_cast<float4*>(out + static_cast<long long>(list) * P.L_stride + pos) = acc;
  // the search kernel's CTAs may move in as this grid drains (earlier, they would take thread
  // slots from CTAs that still stream); it waits for the whole grid before reading a[]
  pdl_launch_dependents();
}

// Number of index lists of a call (0 on invalid arguments) -- shared by the entry point and
// the workspace query.
long long count_lists(const specattn_select_args& A) {
  if (A.n_draft_layers < 1 || A.n_draft_layers > SPECATTN_MAX_DRAFT_LAYERS || A.n_target_layers < 0 ||
      A.batch < 0 || A.n_groups < 1 || A.layer_map == nullptr)
    return 0;
  bool used[SPECATTN_MAX_DRAFT_LAYERS] = {false};
  int n_used = 0;
  for (int j = 0; j < A.n_target_layers; ++j) {
    const int u = A.layer_map[j];
    if (u < -1 || u >= A.n_draft_layers) return 0;
    if (u >= 0 && !used[u]) {
      used[u] = true;
      ++n_used;
    }
  }
  return static_cast<long long>(n_used) * A.batch * A.n_groups;
}

int pick_cluster(long long L_stride, long long n_lists) {
  int cs = 1;
  while (cs < 8 && (L_stride + cs - 1) / cs > 8192) cs *= 2;
  while (cs < 8 && n_lists * cs < 296 && L_stride / cs > 2048) cs *= 2;
  return cs;
}

// The two-launch form applies to the default selection over multi-row lists of >= 2048
// positions, and pays when one cluster per list would leave SMs without a CTA: a CTA streams
// ~35 GB/s, so the cluster kernel is bound by (bytes per list) / (8 x 35 GB/s) however few the
// lists, while the search launch adds ~25 us of its own.  Measured (us, cluster / two-launch):
// 4 lists x 64 rows x 131072: 121 / 94; 16 such lists: 237 / 152; 32 lists x 60 rows x 32768
// (256 CTAs): 71 / 94.
bool two_launch_shape(const specattn_select_args& A) {
  const bool variant = (A.per_step && A.gamma > 1) || A.bisect_iters > 0 || A.chunk > 1;
  if (variant || static_cast<long long>(A.n_draft_heads) * A.gamma <= 1 || A.L_stride < 2048 || A.L_stride % 4 != 0)
    return false;
  const long long n_lists = count_lists(A);
  if (n_lists <= 0 || A.form == SPECATTN_SELECT_FORM_CLUSTER) return false;
  if (A.form == SPECATTN_SELECT_FORM_TWO_LAUNCH) return true;  // the caller knows its batch (ragged lengths)
  return n_lists * pick_cluster(A.L_stride, n_lists) < 148;
}

}  // namespace
}  // namespace specattn

using specattn::SelectParams;

extern "C" size_t specattn_select_workspace_bytes(const specattn_select_args* args) {
  if (args == nullptr || args->struct_size != sizeof(specattn_select_args)) return 0;
  if (!specattn::two_launch_shape(*args)) return 0;
  return static_cast<size_t>(specattn::count_lists(*args)) * static_cast<size_t>(args->L_stride) * sizeof(float);
}

extern "C" int specattn_select_topp(const specattn_select_args* args, void* cuda_stream) {
  specattn::NvtxRange nvtx_range("specattn_select_topp");
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
  if (A.bisect_iters < 0 || A.bisect_iters > 64 || (A.per_step != 0 && A.per_step != 1)) return SPECATTN_ERR_RANGE;
  if (A.form < 0 || A.form > SPECATTN_SELECT_FORM_TWO_LAUNCH) return SPECATTN_ERR_RANGE;
  if (A.chunk < 0 || A.chunk > 64 || (A.chunk > 1 && (A.chunk < 4 || (A.chunk & (A.chunk - 1)) != 0)))
    return SPECATTN_ERR_RANGE;  // 0 / 1 = per position, else a power of two in [4, 64]
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
      if (A.head_group[h] > 127) return SPECATTN_ERR_UNSUPPORTED;
      P.head_group[h] = static_cast<signed char>(A.head_group[h]);
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

  // single-row lists are read in place once the rows are long enough for the extra CTAs per
  // SM to pay for re-reading them from L2 (measured cross-over between 8k and 64k positions)
  P.single_row = (static_cast<long long>(A.n_draft_heads) * A.gamma == 1 && A.L_stride >= 2048) ? 1 : 0;
  // two-launch form: the rows are summed into the workspace first and the search reads that sum
  // in place like a single-row list
  const bool two_launch = A.workspace != nullptr && specattn::two_launch_shape(A) &&
                          A.workspace_bytes >= static_cast<uint64_t>(n_lists) * A.L_stride * sizeof(float);
  if (two_launch) {
    if (reinterpret_cast<uintptr_t>(A.workspace) % 16 != 0) return SPECATTN_ERR_ALIGN;
    P.single_row = 1;
    P.agg = static_cast<const float*>(A.workspace);
  }
  P.per_step = (A.per_step && A.gamma > 1) ? 1 : 0;  // with one query the union is the single nucleus
  P.bisect_iters = A.bisect_iters;
  P.chunk = (A.chunk > 1) ? A.chunk : 1;
  if (P.chunk > 1) P.single_row = 0;  // chunk scores live in the shared-memory slice
  const bool variant = P.per_step || P.bisect_iters > 0 || P.chunk > 1;
  int cs = specattn::pick_cluster(A.L_stride, n_lists);
  if (P.single_row) {
    // A row read in place needs no shared-memory slice, so the cluster only has to keep a slice
    // below 2^16 positions (the 16-bit halves of the mantissa sums must not wrap) and to fill
    // the GPU: with hundreds of rows, one or two CTAs per row avoid most cluster barriers
    // (measured: 256 rows of 8k in one CTA each 31 us against 45 us as pairs; rows of 64k are
    // faster as pairs, 126 us against 152 us).
    cs = 1;
    while (cs < 8 && (A.L_stride + cs - 1) / cs > 65536) cs *= 2;
    while (cs < 8 && n_lists * cs < 296 && (A.L_stride + cs - 1) / cs > 16384) cs *= 2;
    while (cs < 8 && n_lists * cs < 148 && (A.L_stride + cs - 1) / cs > 2048) cs *= 2;  // (short rows: fewer cluster barriers beat more CTAs)
  }
  const long long s_align = (P.chunk > 4) ? P.chunk : 4;
  const long long slice = P.single_row ? 0 : (((A.L_stride + cs - 1) / cs) + s_align - 1) / s_align * s_align;
  if (slice > specattn::kSliceCap) return SPECATTN_ERR_UNSUPPORTED;
  // shared memory: fixed part, the aggregated slice, then the per-thread staging ring
  // (kDepth pieces of 8 KB; it later hosts the scan arrays).  Small slices leave room for two
  // CTAs per SM.
  const size_t fixed = ((sizeof(specattn::Shared) + 127) / 128) * 128 +
                       (P.single_row ? 0 : SPECATTN_MAX_ROWS_PER_LIST * sizeof(long long));
  const size_t slice_bytes = static_cast<size_t>((slice + 31) / 32 * 32) * sizeof(float);
  // (a single-row list keeps nothing but the 32 KB of scan arrays behind the fixed part)
  const size_t smem = fixed + slice_bytes +
                      (P.single_row ? static_cast<size_t>(32 * 1024) : static_cast<size_t>(specattn::kRingFloats) * sizeof(float)) +
                      // the union's bit mask: one bit per position of the slice (sized to the slice, not
                      // to the largest one: with 3 KB for it two CTAs no longer fitted an SM on 32k rows)
                      (P.per_step ? static_cast<size_t>((slice + 127) / 128 * 16) : 0);
  if (smem > 224 * 1024) return SPECATTN_ERR_UNSUPPORTED;
  // Opt in to large dynamic shared memory once per device, so that later calls issue nothing
  // but the launch.
  cudaError_t err = cudaSuccess;
  {
    static std::atomic<unsigned long long> done_mask{0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPECATTN_ERR_CUDA;
    if (!((done_mask.load(std::memory_order_acquire) >> dev) & 1ull)) {
      err = cudaFuncSetAttribute(specattn::select_topp_kernel<false, false>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
      if (err == cudaSuccess)
        err = cudaFuncSetAttribute(specattn::select_topp_kernel<true, false>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
      if (err == cudaSuccess)
        err = cudaFuncSetAttribute(specattn::select_topp_kernel<false, true>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
      if (err == cudaSuccess)
        err = cudaFuncSetAttribute(specattn::select_topp_kernel<true, true>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
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
  cfg.blockDim = dim3(specattn::kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = static_cast<cudaStream_t>(cuda_stream);
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(cs);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (two_launch) {
    const dim3 grid(static_cast<unsigned>((A.L_stride + specattn::kAggPositions - 1) / specattn::kAggPositions),
                    static_cast<unsigned>(n_lists), 1);
    specattn::aggregate_rows_kernel<<<grid, specattn::kAggThreads, 0, cfg.stream>>>(P, static_cast<float*>(A.workspace));
    if (cudaGetLastError() != cudaSuccess) return SPECATTN_ERR_CUDA;
    specattn::g_launch_count.fetch_add(1, std::memory_order_relaxed);
    // the search may be scheduled while the aggregation drains; it waits before reading a[]
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 2;
  }
  // Few clusters: ask for more shared memory than needed, so that an SM takes fewer CTAs and the
  // clusters spread over the GPU instead of filling every slot of a few SMs (co-resident CTAs
  // slow one another's passes: 32 CTAs took 79 us packed, 62 us spread) -- but only as far as
  // all clusters still run at once (clusters are placed GPC by GPC; 16 clusters of 8 do not fit
  // at one CTA per SM, and a second wave costs far more).  The limits are asked of the runtime
  // once per cluster size and cached.
  {
    const void* fn = variant ? (P.single_row ? (const void*)specattn::select_topp_kernel<true, true>
                                             : (const void*)specattn::select_topp_kernel<false, true>)
                             : (P.single_row ? (const void*)specattn::select_topp_kernel<true, false>
                                             : (const void*)specattn::select_topp_kernel<false, false>);
    static const size_t pads[3] = {120 * 1024, 100 * 1024, 70 * 1024};
    static std::atomic<int> fit[64][4][4][3];  // [device][kernel][log2 cs][pad]: clusters + 1, 0 = unknown
    int dev = 0;
    cudaGetDevice(&dev);
    const int kidx = (variant ? 2 : 0) + (P.single_row ? 1 : 0);
    int lcs = 0;
    while ((1 << lcs) < cs) ++lcs;
    for (int k = 0; k < 3 && dev >= 0 && dev < 64; ++k) {
      if (pads[k] <= smem) break;
      int known = fit[dev][kidx][lcs][k].load(std::memory_order_relaxed);
      if (known == 0) {
        cudaLaunchConfig_t q = cfg;
        q.dynamicSmemBytes = pads[k];
        q.gridDim = dim3(static_cast<unsigned>(cs), 1024, 1);
        int n_fit = 0;
        if (cudaOccupancyMaxActiveClusters(&n_fit, fn, &q) != cudaSuccess) {
          cudaGetLastError();
          n_fit = 0;
        }
        known = n_fit + 1;
        fit[dev][kidx][lcs][k].store(known, std::memory_order_relaxed);
      }
      if (known - 1 >= n_lists) {
        cfg.dynamicSmemBytes = pads[k];
        break;
      }
    }
  }
  if (variant)
    err = P.single_row ? cudaLaunchKernelEx(&cfg, specattn::select_topp_kernel<true, true>, P)
                       : cudaLaunchKernelEx(&cfg, specattn::select_topp_kernel<false, true>, P);
  else
    err = P.single_row ? cudaLaunchKernelEx(&cfg, specattn::select_topp_kernel<true, false>, P)
                       : cudaLaunchKernelEx(&cfg, specattn::select_topp_kernel<false, false>, P);
  if (err != cudaSuccess) {
    cudaGetLastError();
    return SPECATTN_ERR_CUDA;
  }
  specattn::g_launch_count.fetch_add(1, std::memory_order_relaxed);
  return SPECATTN_OK;
}
