// sparse_verify on the 5th-generation tensor cores (tcgen05) -- included by sparse_verify.cu
// inside namespace specattn::{anonymous}; shares VerifyParams, the work partition and the
// cross-CTA merge protocol with the mma.sync kernel there.
//
// Same operation (Eq. 1 over the listed rows, Sec. 3.5 / Alg. 1 "Verification with Sparse
// Attention").  The query block of a unit has at most 64 rows, far fewer than the 128 rows a
// tcgen05.mma produces, so both products are computed TRANSPOSED: the 128 KEYS of a tile (or
// the 128 output dimensions) are the M side of the instruction, the N = 16..64 query rows its
// N side:
//   S^T[128 keys x N]  = K[128 x 128] Q^T          A = K tile, B = Q tile, both K-major in smem
//   O^T[128 dims x N] += V^T[128 x 128 keys] P^T   A = V tile (MN-major), B = P^T (MN-major)
// No tensor work is spent on padding rows, and -- because a TMEM lane is a key (or an output
// dimension) -- the softmax warps are spread over the four lane quadrants, i.e. over the four SM
// sub-partitions: a warp owns 32 keys of every tile (and half of the query rows).  P = exp2(S - m) is written as two bf16
// terms (P = P_hi + P_lo) into the shared-memory bytes of the K tile it was computed from,
// which are dead once S^T is complete; the stage is released when the P V product has read it.
//
// The reference maximum m of a row is raised lazily: a tile whose scaled scores stay below
// m + 8 (in the log2 domain) is exponentiated against the old m (P < 2^8, exact enough in two
// bf16 terms and fp32 accumulation); only a tile that exceeds it takes the slow path (row
// maxima over the 128 keys by warp butterflies and a small shared-memory exchange, then a
// rescale of the O^T columns in tensor memory).  Whether a tile takes it is agreed per tile
// through one named barrier of the softmax warps.
//
// Page-granular calls (kPaged: dense calls, and lists made of whole aligned 16-position chunks, on
// caches whose page size is a multiple of 16): a 16-token atom of a unit is 16 consecutive slots
// of one page, i.e. a regular [16 slots x 64 elements] box of the K/V pool for each 128-byte half
// of the head dimension.  Those tiles are fetched with tiled bulk tensor copies (TMA, 128-byte
// swizzle: exactly the operand layout above, completion counted in bytes on the stage's barrier)
// -- four requests per atom instead of 512 16-byte copies, no per-thread addresses, no proxy
// fence.  Half tiles that hold in-flight tokens behind a list, or a list's cut last chunk, take
// the per-row path.
//
// Warps: 0-7 softmax (TMEM lane quadrant = warp % 4, half of the query rows = warp / 4, so every
// SM sub-partition runs two of them), 8 = MMA issue (one thread), 9-12 = producers: two warps per tile, 64 keys each, 16-byte cp.async straight into the
// 128-byte-swizzled operand layout, then fence.proxy.async before the arrival.
#pragma once

constexpr int kTcTile = 128;                     // keys per tile
constexpr int kTcTileBytes = kTcTile * 256;      // one K or V tile (32 KB)
constexpr int kTcStages = 3;
constexpr int kTcRec = 130 * 32;                 // floats of a record per 32 query rows
constexpr float kTcRaise = 8.f;                  // raise the reference maximum beyond 2^8
constexpr int kTcThreads = 13 * 32;
constexpr int kTcMmaWarp = 8;
constexpr int kTcSoftmaxThreads = 256;

// byte offset of 16-byte chunk `c` (0..15) of row `r` in a tile of `rows` rows of 256 bytes: two
// 128-byte halves per row, chunks XOR-swizzled with the row index (UMMA 128-byte swizzle)
__device__ __forceinline__ uint32_t tc_sw(int r, int c, int rows) {
  return static_cast<uint32_t>((c >> 3) * rows * 128 + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr >> 4) & 0x3FFFu);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;  // descriptor version of sm_100
  d |= 2ull << 61;  // 128-byte swizzle
  return d;
}
// instruction descriptor: bf16 x bf16 -> f32, M x N, operand majorness (0 = K, 1 = MN)
__device__ __forceinline__ uint32_t tc_idesc(int M, int N, int a_major, int b_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a_major) << 15) |
         (static_cast<uint32_t>(b_major) << 16) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}" ::"r"(d_tmem),
      "l"(a), "l"(b), "r"(idesc), "r"(acc), "r"(0u)
      : "memory");
}
// arrival on an mbarrier once every tcgen05 operation issued so far by this thread has completed
__device__ __forceinline__ void tc_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// One box of a 5-D tiled tensor map (element, head, slot, k/v, page) into shared memory; bytes are
// counted on `bar`.  No multicast; x (c0) is 0 or 64 elements, i.e. a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_5d(uint32_t dst_smem, const CUtensorMap* map, unsigned long long* bar, int c0,
                                            int c1, int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::
          "r"(dst_smem),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
// The same box, only as far as L2 (no destination, no completion to wait for).
__device__ __forceinline__ void tma_prefetch_5d(const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4) {
  asm volatile("cp.async.bulk.prefetch.tensor.5d.L2.global.tile [%0, {%1, %2, %3, %4, %5}];" ::"l"(
                   reinterpret_cast<uint64_t>(map)),
               "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 lanes x 16 columns of 32 bits: thread t of the warp gets / provides TMEM lane (base + t)
__device__ __forceinline__ void tc_ld16(uint32_t (&r)[16], uint32_t addr) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(addr));
}
__device__ __forceinline__ void tc_st16(uint32_t addr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(
          addr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tc_ld8(uint32_t (&r)[8], uint32_t addr) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(addr));
}
__device__ __forceinline__ void tc_st8(uint32_t addr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(addr), "r"(r[0]),
               "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
// named barrier that also ORs a predicate over its participants: everyone gets the same answer,
// so a group that must leave together can decide to leave on it
__device__ __forceinline__ bool named_bar_or(int id, int nthreads, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %3, 0;\n\t"
      "barrier.red.or.pred q, %1, %2, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"(id), "r"(nthreads), "r"(static_cast<uint32_t>(pred))
      : "memory");
  return r != 0;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  // (no memory clobber: the target bytes are only ever touched through such stores and by the
  // tensor core, and ordinary loads may move across them; the proxy fence that follows orders them)
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d));
}

__device__ __forceinline__ void tc_lds16(float (&d)[16], const float* p) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float4 v = reinterpret_cast<const float4*>(p)[i];
    d[4 * i] = v.x; d[4 * i + 1] = v.y; d[4 * i + 2] = v.z; d[4 * i + 3] = v.w;
  }
}
__device__ __forceinline__ void tc_lds16(int (&d)[16], const int* p) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int4 v = reinterpret_cast<const int4*>(p)[i];
    d[4 * i] = v.x; d[4 * i + 1] = v.y; d[4 * i + 2] = v.z; d[4 * i + 3] = v.w;
  }
}

__device__ __forceinline__ void tc_lds8(float (&d)[8], const float* p) {
  const float4 v0 = reinterpret_cast<const float4*>(p)[0], v1 = reinterpret_cast<const float4*>(p)[1];
  d[0] = v0.x; d[1] = v0.y; d[2] = v0.z; d[3] = v0.w; d[4] = v1.x; d[5] = v1.y; d[6] = v1.z; d[7] = v1.w;
}
__device__ __forceinline__ void tc_lds8(int (&d)[8], const int* p) {
  const int4 v0 = reinterpret_cast<const int4*>(p)[0], v1 = reinterpret_cast<const int4*>(p)[1];
  d[0] = v0.x; d[1] = v0.y; d[2] = v0.z; d[3] = v0.w; d[4] = v1.x; d[5] = v1.y; d[6] = v1.z; d[7] = v1.w;
}

// Butterfly reduce-scatter over the 32 lanes of a warp: v[i] is this lane's value for row i;
// afterwards lane r holds the reduction of row r (returned).  31 shuffles.
template <bool kMax>
__device__ __forceinline__ float tc_reduce_scatter(float (&v)[32], int lane) {
#pragma unroll
  for (int step = 16; step >= 1; step >>= 1) {
    const bool upper = (lane & step) != 0;
#pragma unroll
    for (int i = 0; i < step; ++i) {
      const float send = upper ? v[i] : v[i + step];
      const float keep = upper ? v[i + step] : v[i];
      const float recv = __shfl_xor_sync(0xffffffffu, send, step);
      v[i] = kMax ? fmaxf(keep, recv) : (keep + recv);
    }
  }
  return v[0];
}

struct TcShared {
  alignas(1024) unsigned char kv[kTcStages][2 * kTcTileBytes];  // per stage: K tile (later P^T), V tile
  alignas(1024) unsigned char q[64 * 256];
  alignas(16) float m_ref[64];     // reference maximum of every query row (scaled log2 domain)
  alignas(16) float alpha[64];     // rescale factors of the tile that raised it
  alignas(16) float lsum[64];      // row sums at the end of a unit
  float wred[4][64];   // per-warp row maxima / row sums
  int row_off[64];     // query row r -> t * Hq + (r % grp): its output row inside (b, kv head)
  alignas(16) int row_lim[64];     // last in-flight token row r may see
  alignas(8) unsigned long long full[kTcStages];
  unsigned long long empty[kTcStages];
  unsigned long long q_full, q_empty;
  unsigned long long s_full[2], s_free[2], p_full[2], pv_done[2], o_free;
  uint32_t tmem_base;
  int raise_tile[2];   // tile index + 1 of the last tile (per S buffer) that must raise m_ref
  int last_arriver;
  int unit_start[kMaxUnits + 1];
  int part_start[kAlignedMaxUnits + 1];
  int cand_parts[kCandidates];
  int cand_max[kCandidates];
  volatile int abort_flag;
};

// NT = N / 16, N = query rows rounded up to a multiple of 16
template <int NT, bool kPaged>
__global__ void __launch_bounds__(kTcThreads, 1) sparse_verify_tc_kernel(const __grid_constant__ VerifyParams P,
                                                                       const __grid_constant__ CUtensorMap kv_map) {
  constexpr int N = NT * 16;
  constexpr int NS = kTcStages;
  constexpr int NTH = kTcThreads;
  constexpr int NBLK = (N + 31) / 32;
  extern __shared__ __align__(1024) unsigned char smem_raw_tc[];
  TcShared& sh =
      *reinterpret_cast<TcShared*>((reinterpret_cast<uintptr_t>(smem_raw_tc) + 1023) & ~static_cast<uintptr_t>(1023));
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const int U = P.B * P.Hkv;

  if (!P.lists_stable) pdl_wait();
  pdl_launch_dependents();

  // ---- set-up ---------------------------------------------------------------------------------
  {
    uint4* zq = reinterpret_cast<uint4*>(sh.q);  // rows beyond the query block stay zero
    for (int i = tid; i < static_cast<int>(sizeof(sh.q) / 16); i += NTH) zq[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&sh.full[s], 2);   // two producer warps per tile
      mbar_init(&sh.empty[s], 1);
    }
    mbar_init(&sh.q_full, 1);
    mbar_init(&sh.q_empty, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sh.s_full[i], 1);
      mbar_init(&sh.s_free[i], 8);   // one arrival per softmax warp
      mbar_init(&sh.p_full[i], 8);
      mbar_init(&sh.pv_done[i], 1);
    }
    mbar_init(&sh.o_free, 8);
    mbar_fence_init();
    sh.abort_flag = 0;
    sh.raise_tile[0] = sh.raise_tile[1] = 0;
    sh.unit_start[0] = 0;
  }
  if (tid < 64) {
    sh.row_off[tid] = (tid / P.grp) * P.Hq + tid % P.grp;
    sh.row_lim[tid] = tid / P.grp + P.tail_off;
  }
  for (int u = tid; u < U; u += NTH) sh.unit_start[u + 1] = (unit_count(P, u) + kAtom - 1) / kAtom;
  fence_proxy_async();
  __syncthreads();
  if (warp == 0) {  // inclusive scan of the atom counts
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

  // ---- work partition (the two schemes of the mma.sync kernel) -----------------------------------
  const long long NA = sh.unit_start[U];
  const int G = static_cast<int>(gridDim.x);
  if (tid < kCandidates) { sh.cand_parts[tid] = 0; sh.cand_max[tid] = 0; }
  __syncthreads();
  const bool try_aligned = (U <= kAlignedMaxUnits) && (NA > 0);
  if (try_aligned && tid < U) {
    const int atoms = sh.unit_start[tid + 1] - sh.unit_start[tid];
    if (atoms > 0) {
#pragma unroll
      for (int c = 0; c < kCandidates; ++c) {
        const long long num = static_cast<long long>(atoms) * G * 16;
        const long long den = NA * (16 + c);
        int k = static_cast<int>((2 * num + den) / (2 * den));
        if (k < 1) k = 1;
        if (k > atoms) k = atoms;
        if (k * kMinPartAtoms > atoms) k = max(1, atoms / kMinPartAtoms);  // no part shorter than that
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
    if (cand >= 0 && static_cast<long long>(sh.cand_max[cand]) * G > NA + 24ll * G) cand = -1;
  }
  const bool aligned = cand >= 0;
  if (aligned && warp == 0) {
    int carry = 0;
    for (int base = 0; base < U; base += 32) {
      const int u = base + lane;
      int k = 0;
      if (u < U) {
        const int atoms = sh.unit_start[u + 1] - sh.unit_start[u];
        if (atoms > 0) {
          const long long num = static_cast<long long>(atoms) * G * 16;
          const long long den = NA * (16 + cand);
          k = static_cast<int>((2 * num + den) / (2 * den));
          if (k < 1) k = 1;
          if (k > atoms) k = atoms;
        if (k * kMinPartAtoms > atoms) k = max(1, atoms / kMinPartAtoms);  // no part shorter than that
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
  const long long NP = aligned ? sh.part_start[U] : ((NA < G) ? NA : static_cast<long long>(G));

  const bool is_softmax = warp < 8;
  const bool is_mma = (warp == kTcMmaWarp);
  // The softmax warps are the only ones that write global memory; with SPECATTN_VERIFY_LISTS_STABLE
  // they wait for the previous kernel here.  (For a CTA that gets work this comes after the
  // tensor-memory allocation and the barrier behind it: the producers must not be held up by
  // that wait -- their copies are what may run under the previous kernel.)
  auto wait_and_clear_empty_units = [&]() {
    if (P.lists_stable) pdl_wait();  // (otherwise the whole kernel has waited at its start)
    // units with an empty list: out = 0, lse = -inf
    for (int u = blockIdx.x; u < U; u += gridDim.x) {
      if (unit_count(P, u) != 0) continue;
      const int b = u / P.Hkv, kvh = u % P.Hkv;
      for (int e = tid; e < P.M * kD; e += kTcSoftmaxThreads) {
        const int r = e / kD, t = r / P.grp, h = kvh * P.grp + r % P.grp;
        P.out[((static_cast<long long>(b) * P.T + t) * P.Hq + h) * kD + e % kD] = 0.f;
        if (e % kD == 0) P.lse[(static_cast<long long>(b) * P.T + t) * P.Hq + h] = -INFINITY;
      }
    }
  };
  if (is_softmax && !P.lists_stable) wait_and_clear_empty_units();  // nothing to wait for: do it now
  if (static_cast<long long>(blockIdx.x) >= NP) {
    if (is_softmax && P.lists_stable) wait_and_clear_empty_units();
    return;
  }
  int a0, a1;
  if (aligned) {
    int lo = 0, hi = U - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (sh.part_start[mid] <= static_cast<int>(blockIdx.x)) lo = mid; else hi = mid - 1;
    }
    const int k = sh.part_start[lo + 1] - sh.part_start[lo];
    const int j = static_cast<int>(blockIdx.x) - sh.part_start[lo];
    const long long atoms = sh.unit_start[lo + 1] - sh.unit_start[lo];
    a0 = sh.unit_start[lo] + static_cast<int>(j * atoms / k);
    a1 = sh.unit_start[lo] + static_cast<int>((j + 1) * atoms / k);
  } else {
    a0 = cta_first_atom(blockIdx.x, NA, NP);
    a1 = cta_first_atom(blockIdx.x + 1, NA, NP);
  }
  int u_first;
  {
    int lo = 0, hi = U - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (sh.unit_start[mid] <= a0) lo = mid; else hi = mid - 1;
    }
    u_first = lo;
    while (sh.unit_start[u_first + 1] <= a0) ++u_first;
  }

  // ---- tensor memory: S^T double-buffered (N columns each), O^T (2 N: P_hi and P_lo parts) ------
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)),
                 "r"(256u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;
  const uint32_t col_o = tmem + 2u * N;  // 2 N columns: the P_hi part, then the P_lo part
  if (is_softmax && P.lists_stable) wait_and_clear_empty_units();

  auto next_unit = [&](int& a, int& u, int seg_hi, int ue) {
    a = seg_hi;
    if (a == ue) {
      ++u;
      while (u < U && sh.unit_start[u + 1] == sh.unit_start[u]) ++u;
    }
  };

  if (!is_softmax && !is_mma) {
    // =============================== producer warps ===============================================
    // tile i is filled by warps 2 (i & 1) and 2 (i & 1) + 1: keys 0..63 and 64..127 of the tile
    const int pw = warp - 9;
    const int tpar = pw >> 1, half = pw & 1;
    int it = 0, seg = 0;
    int a = a0, u = u_first;
    bool dead = false;
    while (a < a1 && !dead) {
      const int us = sh.unit_start[u], ue = sh.unit_start[u + 1];
      const int seg_hi = min(a1, ue);
      const int b = u / P.Hkv, kvh = u % P.Hkv;
      const int ucnt = unit_count(P, u);
      const int tok_lo = (a - us) * kAtom;
      const int tok_hi = min(ucnt, (seg_hi - us) * kAtom);
      const int kvlen_b = P.kv_len[b];
      const int c_list = ucnt - P.tail;
      const int* list = P.dense ? nullptr
                                : P.idx + (static_cast<long long>(b) * P.G + ((P.G == 1) ? 0 : kvh)) * P.idx_stride;
      const __nv_bfloat16* kv_head = P.kv + static_cast<long long>(kvh) * P.s_head;
      // The query block of this unit, straight into the swizzled operand layout; always by
      // producer warp 0, walking the segments in order (for the first segment after the warp's
      // first half tile, so that K/V prefetch is in flight while it waits for the previous kernel).
      auto load_q = [&]() -> bool {
        if (seg == 0 && P.lists_stable) pdl_wait();
        if (!mbar_wait(&sh.q_empty, (seg & 1u) ^ 1u, &sh.abort_flag)) return false;
        const uint32_t qb = smem_u32(sh.q);
        for (int i = lane; i < P.M * 16; i += 32) {
          const int r = i >> 4, c = i & 15;
          const int t = r / P.grp, h = kvh * P.grp + r % P.grp;
          cp_async16(qb + tc_sw(r, c, 64), P.q + ((static_cast<long long>(b) * P.T + t) * P.Hq + h) * kD + c * 8);
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.q_full);
        return true;
      };
      bool q_pending = (pw == 0);
      if (q_pending && seg > 0) {
        q_pending = false;
        if (!load_q()) { sh.abort_flag = 1; dead = true; break; }
      }
      // lane j resolves keys j and j + 32 of this warp's half tile to the byte offset of their K row
      auto resolve = [&](int h0, long long (&off)[2]) -> bool {
        const int ntok = min(64, tok_hi - h0);
        bool bad = false;
        if (ntok <= 0) return false;
#pragma unroll
        for (int jj = 0; jj < 2; ++jj) {
          const int jt = min(lane + jj * 32, ntok - 1);
          const int k = h0 + jt;  // token index inside the unit: the list first, then the tail
          int pos = (k >= c_list) ? (kvlen_b + (k - c_list)) : (P.dense ? k : __ldg(list + k));
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
      // (page-granular) lane j < 4 resolves atom j of this warp's half tile to (page, first slot),
      // packed as page * 4096 + slot; one list entry and one block-table entry per 16 tokens
      const int c_list16 = c_list & ~15;
      auto tma_half = [&](int h0) -> bool {
        return kPaged && (P.dense || min(h0 + 64, tok_hi) <= c_list16);
      };
      auto resolve_atom = [&](int h0, long long& where) -> bool {
        bool bad = false;
        where = 0;
        const int k = h0 + 16 * lane;
        if (lane < 4 && k < tok_hi) {
          int pos = P.dense ? k : __ldg(list + k);
          if (pos < 0 || pos >= kvlen_b + P.tail || (pos & 15)) { bad = true; pos = 0; }
          int lp = (P.page_shift >= 0) ? (pos >> P.page_shift) : (pos / P.page_size);
          if (lp >= P.bt_stride) { bad = true; pos = 0; lp = 0; }
          const int slot = pos - lp * P.page_size;
          long long page = P.bt ? static_cast<long long>(__ldg(P.bt + b * P.bt_stride + lp))
                                : (b * P.bt_stride + lp);
          if (page < 0 || page >= P.n_pages) { bad = true; page = 0; }
          where = page * 4096 + slot;
        }
        return bad;
      };
      long long off_next[2] = {0, 0};
      bool bad_next = false;
      int t0_next = -1;
      for (int t0 = tok_lo; t0 < tok_hi; t0 += kTcTile, ++it) {
        if ((it & 1) != tpar) continue;
        const int s = it % NS;
        const unsigned ph = (it / NS) & 1u;
        const int h0 = t0 + half * 64;
        if (tma_half(h0)) {
          long long where;
          bool bad;
          if (t0_next == t0) {
            where = off_next[0];
            bad = bad_next;
          } else {
            bad = resolve_atom(h0, where);
          }
          t0_next = t0 + 2 * kTcTile;
          if (t0_next < tok_hi && tma_half(t0_next + half * 64)) {
            // this warp's next half tile: resolved now, and its boxes asked into L2 at once -- two
            // tiles ahead of the ring, so that the copies into shared memory find them there
            bad_next = resolve_atom(t0_next + half * 64, off_next[0]);
            const int hn = t0_next + half * 64;
            if (lane < 4 && hn + 16 * lane < tok_hi) {
              const int page = static_cast<int>(off_next[0] >> 12), slot = static_cast<int>(off_next[0] & 4095);
              tma_prefetch_5d(&kv_map, 0, kvh, slot, 0, page);
              tma_prefetch_5d(&kv_map, 64, kvh, slot, 0, page);
              tma_prefetch_5d(&kv_map, 0, kvh, slot, 1, page);
              tma_prefetch_5d(&kv_map, 64, kvh, slot, 1, page);
            }
          } else {
            t0_next = -1;
          }
          if (!mbar_wait(&sh.empty[s], ph ^ 1u, &sh.abort_flag)) { sh.abort_flag = 1; dead = true; break; }
          const int ntok = max(0, min(64, tok_hi - h0));
          const int natoms = (ntok + 15) >> 4;
          if (lane == 0) {
            // 4 boxes of 2 KB per atom: K and V, two 128-byte halves of the head dimension each
            if (natoms > 0) mbar_arrive_expect_tx(&sh.full[s], static_cast<uint32_t>(natoms) * 4u * 2048u);
            else mbar_arrive(&sh.full[s]);
          }
          __syncwarp();
          if (lane < natoms) {
            const int page = static_cast<int>(where >> 12), slot = static_cast<int>(where & 4095);
            const uint32_t k_dst = smem_u32(sh.kv[s]) + (half * 64 + 16 * lane) * 128;
            const uint32_t v_dst = k_dst + kTcTileBytes;
            tma_load_5d(k_dst, &kv_map, &sh.full[s], 0, kvh, slot, 0, page);
            tma_load_5d(k_dst + kTcTile * 128, &kv_map, &sh.full[s], 64, kvh, slot, 0, page);
            tma_load_5d(v_dst, &kv_map, &sh.full[s], 0, kvh, slot, 1, page);
            tma_load_5d(v_dst + kTcTile * 128, &kv_map, &sh.full[s], 64, kvh, slot, 1, page);
          }
          if (__any_sync(0xffffffffu, bad) && P.status && lane == 0) atomicOr(P.status + b, SPECATTN_ROW_BAD_INDEX);
          if (q_pending) {
            q_pending = false;
            if (!load_q()) { sh.abort_flag = 1; dead = true; break; }
          }
          continue;
        }
        long long off[2] = {0, 0};
        bool bad;
        if (t0_next == t0) {
          off[0] = off_next[0];
          off[1] = off_next[1];
          bad = bad_next;
        } else {
          bad = resolve(h0, off);
        }
        t0_next = t0 + 2 * kTcTile;
        if (t0_next < tok_hi && !tma_half(t0_next + half * 64)) bad_next = resolve(t0_next + half * 64, off_next);
        else t0_next = -1;
        if (!mbar_wait(&sh.empty[s], ph ^ 1u, &sh.abort_flag)) { sh.abort_flag = 1; dead = true; break; }
        const int ntok = max(0, min(64, tok_hi - h0));
        const int npad = (ntok + 15) & ~15;  // the P V product runs over whole 16-key steps
        const char* kbase = reinterpret_cast<const char*>(kv_head) + (lane & 15) * 16;
        const long long v_delta = P.s_kv * 2;
        const uint32_t k_dst = smem_u32(sh.kv[s]);
        const uint32_t v_dst = k_dst + kTcTileBytes;
#pragma unroll
        for (int jj = 0; jj < 2; ++jj) {
#pragma unroll 4
          for (int i = 0; i < 16; ++i) {
            const int tok = jj * 32 + 2 * i + (lane >> 4);
            const long long o = __shfl_sync(0xffffffffu, off[jj], 2 * i + (lane >> 4));
            if (tok < npad) {
              const uint32_t d = tc_sw(half * 64 + tok, lane & 15, kTcTile);
              cp_async16(k_dst + d, kbase + o);
              cp_async16(v_dst + d, kbase + o + v_delta);
            }
          }
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
        fence_proxy_async();  // generic-proxy writes -> visible to the tensor core's reads
        __syncwarp();
        // (test hook: the first tile of CTA 0 never completes, so the bounded waits run out)
        if (lane == 0 && !(P.test_lose && blockIdx.x == 0 && it == 0 && half == 0)) mbar_arrive(&sh.full[s]);
        if (bad && P.status) atomicOr(P.status + b, SPECATTN_ROW_BAD_INDEX);
        if (q_pending) {
          q_pending = false;
          if (!load_q()) { sh.abort_flag = 1; dead = true; break; }
        }
      }
      ++seg;
      next_unit(a, u, seg_hi, ue);
    }
    return;
  }

  if (is_mma) {
    // =============================== MMA issue warp (one thread) =================================
    if (lane == 0) {
      const uint32_t idesc = tc_idesc(128, N, 0, 0);      // S^T = K Q^T: both operands K-major
      const uint32_t idesc_pv = tc_idesc(128, 2 * N, 1, 1);  // [O_hi^T | O_lo^T] += V^T [P_hi^T | P_lo^T]
      const uint32_t q_base = smem_u32(sh.q);
      bool ok = true;
      int it = 0, seg = 0;
      int a = a0, u = u_first;
      while (a < a1 && ok) {
        const int us = sh.unit_start[u], ue = sh.unit_start[u + 1];
        const int seg_hi = min(a1, ue);
        const int tok_lo = (a - us) * kAtom;
        const int tok_hi = min(unit_count(P, u), (seg_hi - us) * kAtom);
        const int ntiles = (tok_hi - tok_lo + kTcTile - 1) / kTcTile;
        if (!mbar_wait(&sh.q_full, seg & 1u, &sh.abort_flag)) { ok = false; break; }
        // Issue whichever product is ready: the P V product of the oldest tile that has its P^T
        // (it releases a stage), else S^T of the next tile whose K/V has landed.  Both kinds run
        // in tile order; S^T may lead by the two S buffers.
        int nq = 0, np = 0;  // tiles of this segment whose S^T / P V product has been issued
        bool o_ready = false;
        uint32_t polls = 0;
        while (np < ntiles) {
          bool did = false;
          if (np < nq) {
            const int j = it + np, s = j % NS;
            if (!o_ready) o_ready = (np > 0) || mbar_test(&sh.o_free, (seg & 1u) ^ 1u);
            // per tile parity, like the S buffers: the softmax warps can finish tile j + 1 before
            // this thread looks, and one barrier would then be two phases ahead of the test
            if (o_ready && mbar_test(&sh.p_full[j & 1], (j >> 1) & 1u)) {
              tc_fence_after();
              const int ntok = min(kTcTile, tok_hi - (tok_lo + np * kTcTile));
              const int ksteps = (ntok + 15) >> 4;
              const uint32_t p_base = smem_u32(sh.kv[s]);  // [P_hi^T | P_lo^T] in the K tile's bytes
              const uint32_t v_base = p_base + kTcTileBytes;
              for (int kk = 0; kk < ksteps; ++kk)
                tc_mma_ss(col_o, tc_desc(v_base + kk * 2048, kTcTile * 128, 1024),
                          tc_desc(p_base + kk * 2048, 16384, 1024), idesc_pv, (np == 0 && kk == 0) ? 0u : 1u);
              tc_commit(&sh.empty[s]);
              tc_commit(&sh.pv_done[j & 1]);
              ++np;
              did = true;
            }
          }
          if (!did && nq < ntiles) {
            const int i = it + nq, s = i % NS, sb = i & 1;
            if (mbar_test(&sh.full[s], (i / NS) & 1u) && mbar_test(&sh.s_free[sb], ((i >> 1) & 1u) ^ 1u)) {
              tc_fence_after();
              const uint32_t k_base = smem_u32(sh.kv[s]);
#pragma unroll
              for (int kk = 0; kk < 8; ++kk)
                tc_mma_ss(tmem + sb * N, tc_desc(k_base + (kk >> 2) * (kTcTile * 128) + (kk & 3) * 32, 16, 1024),
                          tc_desc(q_base + (kk >> 2) * (64 * 128) + (kk & 3) * 32, 16, 1024), idesc, kk > 0);
              tc_commit(&sh.s_full[sb]);
              if (nq == ntiles - 1) tc_commit(&sh.q_empty);  // the query tile may be replaced
              ++nq;
              did = true;
            }
          }
          if (did) {
            polls = 0;
          } else {
            if (++polls > (1u << 22) || (polls > 64 && sh.abort_flag)) { ok = false; break; }
            __nanosleep(polls > 4096 ? 100 : 20);  // the issue slots belong to the softmax warp of this sub-partition
          }
        }
        if (!ok) break;
        it += ntiles;
        ++seg;
        next_unit(a, u, seg_hi, ue);
      }
      if (!ok) sh.abort_flag = 1;
    }
    __syncwarp();
  } else {
    // =============================== softmax warps ==============================================
    // warp = (row half, lane quadrant): 32 keys of the tile against half of the query rows
    constexpr int RW = N / 2;   // query rows of this warp
    constexpr int NO = NT;      // ... in groups of eight
    const int quad = warp & 3, r0 = (warp >> 2) * RW;
    const int key_lane = quad * 32 + lane;  // key of the tile / output dimension = TMEM lane
    const uint32_t lane_sel = static_cast<uint32_t>(quad * 32) << 16;
    constexpr int kBar = 1;
    bool fail = false;
    int it = 0, seg = 0;
    // P V products whose completion this thread has seen: every tile is waited for, in order, on
    // the barrier of its parity.  (One barrier for all tiles could complete two phases between
    // two polls -- the product of a short last tile takes a few dozen nanoseconds -- and a
    // parity wait cannot tell that from none.)
    int pv_next = 0;
    auto pv_catch_up = [&](int upto) {
      while (pv_next <= upto) {
        if (!mbar_wait(&sh.pv_done[pv_next & 1], (pv_next >> 1) & 1u, &sh.abort_flag)) { fail = true; return; }
        ++pv_next;
      }
    };
    int a = a0, u = u_first;
    while (a < a1) {
      const int us = sh.unit_start[u], ue = sh.unit_start[u + 1];
      const int seg_hi = min(a1, ue);
      const int b = u / P.Hkv, kvh = u % P.Hkv;
      const int ucnt = unit_count(P, u);
      const int tok_lo = (a - us) * kAtom;
      const int tok_hi = min(ucnt, (seg_hi - us) * kAtom);
      const int c_list = ucnt - P.tail;
      const int ntiles = (tok_hi - tok_lo + kTcTile - 1) / kTcTile;
      if (tid < N) sh.m_ref[tid] = -INFINITY;
      float l_part[RW];
#pragma unroll
      for (int r = 0; r < RW; ++r) l_part[r] = 0.f;
      if (named_bar_or(kBar, kTcSoftmaxThreads, fail)) { fail = true; break; }

      for (int n = 0; n < ntiles; ++n) {
        const int i = it + n, s = i % NS, sb = i & 1;
        const int t0 = tok_lo + n * kTcTile;
        const int ntok = min(kTcTile, tok_hi - t0);
        const bool kvalid = key_lane < ntok;
        // in-flight token index of this key (negative: a listed row, visible to every query)
        const int jt = P.tail ? (key_lane - (c_list - t0)) : -1;
        if (!fail && !mbar_wait(&sh.s_full[sb], (i >> 1) & 1u, &sh.abort_flag)) fail = true;
        tc_fence_after();
        // a tile that holds in-flight tokens masks per (key, query); all others per key only
        const bool tail_tile = P.tail && (t0 + kTcTile > c_list);
        // ---- pass 1: does any visible score exceed its row's reference maximum by 2^8? --------
        bool exceed = false;
        uint32_t sv[NO][8];  // this key's scores against this warp's query rows
        if (!__any_sync(0xffffffffu, fail)) {
#pragma unroll
          for (int o = 0; o < NO; ++o) tc_ld8(sv[o], tmem + sb * N + lane_sel + r0 + o * 8);
          tc_wait_ld();
#pragma unroll
          for (int o = 0; o < NO; ++o) {
            float mr[8];
            tc_lds8(mr, sh.m_ref + r0 + o * 8);
            // from here on sv holds x = s * scale - m, the exponent of P
#pragma unroll
            for (int j = 0; j < 8; ++j)
              sv[o][j] = __float_as_uint(fmaf(__uint_as_float(sv[o][j]), P.scale_log2, -mr[j]));
            if (!tail_tile) {
#pragma unroll
              for (int j = 0; j < 8; ++j) exceed |= !(__uint_as_float(sv[o][j]) <= kTcRaise);
            } else {
              int lim[8];
              tc_lds8(lim, sh.row_lim + r0 + o * 8);
#pragma unroll
              for (int j = 0; j < 8; ++j)
                exceed |= ((jt < 0) | (jt <= lim[j])) & !(__uint_as_float(sv[o][j]) <= kTcRaise);
            }
          }
          exceed &= kvalid;
        }
        if (__any_sync(0xffffffffu, exceed) && lane == 0) sh.raise_tile[sb] = i + 1;
        if (named_bar_or(kBar, kTcSoftmaxThreads, fail)) { fail = true; break; }
        if (sh.raise_tile[sb] == i + 1) {
          // ---- slow path: new row maxima, rescale of the sums and of O^T ----------------------
          {
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = -INFINITY;
            // the raw scores again (the S^T buffer is still this tile's)
#pragma unroll
            for (int o = 0; o < NO; ++o) tc_ld8(sv[o], tmem + sb * N + lane_sel + r0 + o * 8);
            tc_wait_ld();
#pragma unroll
            for (int o = 0; o < NO; ++o) {
              int lim[8];
              tc_lds8(lim, sh.row_lim + r0 + o * 8);
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const bool vis = kvalid & (!tail_tile | (jt < 0) | (jt <= lim[j]));
                v[o * 8 + j] = vis ? __uint_as_float(sv[o][j]) * P.scale_log2 : -INFINITY;
              }
            }
            const float wm = tc_reduce_scatter<true>(v, lane);
            if (lane < RW) sh.wred[quad][r0 + lane] = wm;
          }
          if (named_bar_or(kBar, kTcSoftmaxThreads, fail)) { fail = true; break; }
          if (tid < N) {
            const float mo = sh.m_ref[tid];
            const float mn = fmaxf(fmaxf(mo, sh.wred[0][tid]),
                                   fmaxf(sh.wred[1][tid], fmaxf(sh.wred[2][tid], sh.wred[3][tid])));
            sh.alpha[tid] = (mo == -INFINITY) ? 0.f : ex2(mo - mn);
            sh.m_ref[tid] = mn;
          }
          if (named_bar_or(kBar, kTcSoftmaxThreads, fail)) { fail = true; break; }
          if (n > 0) {  // O^T holds this unit's earlier tiles: quiet once their P V products are done
            pv_catch_up(i - 1);
            tc_fence_after();
            if (!__any_sync(0xffffffffu, fail)) {
#pragma unroll
              for (int c = 0; c < 2 * NO; ++c) {  // this warp's rows in the P_hi and the P_lo part of O^T
                const int col = (c / NO) * N + r0 + (c % NO) * 8;
                uint32_t ov[8];
                tc_ld8(ov, col_o + lane_sel + col);
                float al[8];
                tc_lds8(al, sh.alpha + r0 + (c % NO) * 8);
                tc_wait_ld();
#pragma unroll
                for (int j = 0; j < 8; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * al[j]);
                tc_st8(col_o + lane_sel + col, ov);
              }
              tc_wait_st();
            }
          }
#pragma unroll
          for (int o = 0; o < NO; ++o) {
            float al[8], mr[8];
            tc_lds8(al, sh.alpha + r0 + o * 8);
            tc_lds8(mr, sh.m_ref + r0 + o * 8);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              l_part[o * 8 + j] *= al[j];
              sv[o][j] = __float_as_uint(fmaf(__uint_as_float(sv[o][j]), P.scale_log2, -mr[j]));  // against the new m
            }
          }
        }
        // ---- pass 2: P = exp2(S - m) as two bf16 terms, into the dead K tile ------------------
        if (!__any_sync(0xffffffffu, fail)) {
          const uint32_t pb = smem_u32(sh.kv[s]) + (key_lane >> 3) * 1024 + (key_lane & 7) * 128;
          // every score of this tile is in registers: the S^T buffer may be overwritten
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.s_free[sb]);
#pragma unroll
          for (int o = 0; o < NO; ++o) {
            float p[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) p[j] = ex2(__uint_as_float(sv[o][j]));
            if (tail_tile) {
              int lim[8];
              tc_lds8(lim, sh.row_lim + r0 + o * 8);
#pragma unroll
              for (int j = 0; j < 8; ++j) p[j] = ((jt < 0) | (jt <= lim[j])) ? p[j] : 0.f;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              p[j] = kvalid ? p[j] : 0.f;
              l_part[o * 8 + j] += p[j];
            }
            // P = P_hi + P_lo in bf16 on the integer / FMA pipes: P_hi keeps the upper 16 bits
            // (truncation), P_lo is the exact remainder rounded to nearest (P >= 0, so adding
            // half an ulp to the bit pattern rounds): |P - P_hi - P_lo| <= 2^-16 P, unbiased
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const uint32_t b0 = __float_as_uint(p[2 * e]), b1 = __float_as_uint(p[2 * e + 1]);
              hi[e] = __byte_perm(b0, b1, 0x7632);
              const uint32_t d0 = __float_as_uint(__uint_as_float(b0) - __uint_as_float(b0 & 0xffff0000u)) + 0x8000u;
              const uint32_t d1 = __float_as_uint(__uint_as_float(b1) - __uint_as_float(b1 & 0xffff0000u)) + 0x8000u;
              lo[e] = __byte_perm(d0, d1, 0x7632);
            }
            // B operand [P_hi^T | P_lo^T]: 2N columns, 16-byte chunk ch of a key's row at
            // (ch / 8) * 16 KB + ((ch % 8) ^ (key % 8)) * 16
            const int ch_hi = (r0 >> 3) + o, ch_lo = ch_hi + N / 8;
            st_shared_v4(pb + (ch_hi >> 3) * 16384 + (((ch_hi & 7) ^ (key_lane & 7)) << 4), hi[0], hi[1], hi[2], hi[3]);
            st_shared_v4(pb + (ch_lo >> 3) * 16384 + (((ch_lo & 7) ^ (key_lane & 7)) << 4), lo[0], lo[1], lo[2], lo[3]);
          }
          if (kPaged && warp < 4 && !kvalid && key_lane < ((ntok + 15) & ~15)) {
            // a box copy brought 16 whole slots: those beyond the unit's last token hold whatever
            // the pool holds there (possibly non-finite) and meet P = 0 in the product -- clear them
            const uint32_t vb = smem_u32(sh.kv[s]) + kTcTileBytes;
#pragma unroll
            for (int c = 0; c < 16; ++c) st_shared_v4(vb + tc_sw(key_lane, c, kTcTile), 0u, 0u, 0u, 0u);
          }
          fence_proxy_async();  // P^T is read by the tensor core through the async proxy
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.p_full[sb]);
        }
        if (n > 0 && !fail) pv_catch_up(i - 1);
      }
      if (fail) sh.abort_flag = 1;

      // ---- end of the unit's share: row sums over all keys, O^T out of tensor memory ------------
      {
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = (j < RW) ? l_part[(j < RW) ? j : 0] : 0.f;
        const float ws = tc_reduce_scatter<false>(v, lane);
        if (lane < RW) sh.wred[quad][r0 + lane] = ws;
      }
      if (named_bar_or(kBar, kTcSoftmaxThreads, fail)) { fail = true; break; }
      if (tid < N) sh.lsum[tid] = (sh.wred[0][tid] + sh.wred[1][tid]) + (sh.wred[2][tid] + sh.wred[3][tid]);
      pv_catch_up(it + ntiles - 1);
      tc_fence_after();
      if (named_bar_or(kBar, kTcSoftmaxThreads, fail)) { fail = true; break; }

      const bool whole = (a == us) && (seg_hi == ue);
      const long long obase = static_cast<long long>(b) * P.T * P.Hq + kvh * P.grp;
      const int d = key_lane;  // this thread's output dimension
      if (whole) {
#pragma unroll
        for (int o = 0; o < NO; ++o) {
          uint32_t ov[8], ow[8];
          tc_ld8(ov, col_o + lane_sel + r0 + o * 8);
          tc_ld8(ow, col_o + lane_sel + N + r0 + o * 8);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int r = r0 + o * 8 + j;
            if (r < P.M) {
              const float l = sh.lsum[r];
              P.out[(obase + sh.row_off[r]) * kD + d] =
                  (__uint_as_float(ov[j]) + __uint_as_float(ow[j])) * ((l > 0.f) ? 1.f / l : 0.f);
            }
          }
        }
        if (tid < P.M) {
          const float l = sh.lsum[tid];
          P.lse[obase + sh.row_off[tid]] = (l > 0.f) ? (sh.m_ref[tid] + log2f(l)) * kLn2 : -INFINITY;
        }
      } else {
        // publish this CTA's share ([row][dim] sums, then m, then l), then see who arrived last
        float* rec = P.partials + static_cast<size_t>(2 * blockIdx.x + (a == a0 ? 0 : 1)) * NBLK * kTcRec;
#pragma unroll
        for (int o = 0; o < NO; ++o) {
          uint32_t ov[8], ow[8];
          tc_ld8(ov, col_o + lane_sel + r0 + o * 8);
          tc_ld8(ow, col_o + lane_sel + N + r0 + o * 8);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < 8; ++j)
            __stcg(rec + (r0 + o * 8 + j) * kD + d, __uint_as_float(ov[j]) + __uint_as_float(ow[j]));
        }
        if (tid < N) {
          __stcg(rec + N * kD + tid, sh.m_ref[tid]);
          __stcg(rec + N * kD + N + tid, sh.lsum[tid]);
        }
        __threadfence();
        if (named_bar_or(kBar, kTcSoftmaxThreads, fail)) { fail = true; break; }
        const int i_lo = aligned ? sh.part_start[u] : cta_of_atom(us, NA, NP);
        const int i_hi = aligned ? sh.part_start[u + 1] - 1 : cta_of_atom(ue - 1, NA, NP);
        if (tid == 0) {
          const unsigned int old = atomicAdd(P.counters + u * kCountersPerUnit, 1u);
          sh.last_arriver = (old == static_cast<unsigned int>(i_hi - i_lo)) ? 1 : 0;
        }
        if (named_bar_or(kBar, kTcSoftmaxThreads, fail)) { fail = true; break; }
        if (sh.last_arriver) {
          __threadfence();
          // merge every contributor's record in CTA order, eight query rows at a time
          auto rec_of = [&](int i) {
            return P.partials + static_cast<size_t>(2 * i + ((aligned || cta_first_atom(i, NA, NP) >= us) ? 0 : 1)) *
                                    NBLK * kTcRec;
          };
#pragma unroll 1
          for (int o = 0; o < NO; ++o) {
            // one pass with a running maximum: the 24 loads of a contributor are independent,
            // and two contributors are in flight at a time
            const int rb = r0 + o * 8;
            float mx[8], acc[8], ls[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) { mx[j] = -INFINITY; acc[j] = 0.f; ls[j] = 0.f; }
#pragma unroll 2
            for (int i = i_lo; i <= i_hi; ++i) {
              const float* r2 = rec_of(i);
              float mi[8], li[8], oi[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                mi[j] = __ldcg(r2 + N * kD + rb + j);
                li[j] = __ldcg(r2 + N * kD + N + rb + j);
                oi[j] = __ldcg(r2 + (rb + j) * kD + d);
              }
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                float mn, ao, ai;
                merge_scales(mx[j], mi[j], mn, ao, ai);
                mx[j] = mn;
                ls[j] = ls[j] * ao + li[j] * ai;
                acc[j] = acc[j] * ao + oi[j] * ai;
              }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int r = rb + j;
              if (r < P.M) {
                P.out[(obase + sh.row_off[r]) * kD + d] = acc[j] * ((ls[j] > 0.f) ? 1.f / ls[j] : 0.f);
                if (d == 0) P.lse[obase + sh.row_off[r]] = (ls[j] > 0.f) ? (mx[j] + log2f(ls[j])) * kLn2 : -INFINITY;
              }
            }
          }
          if (tid == 0) P.counters[u * kCountersPerUnit] = 0u;  // ready for the next call
        }
      }
      // O^T may be overwritten by the next unit
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.o_free);
      it += ntiles;
      ++seg;
      next_unit(a, u, seg_hi, ue);
    }
    if (fail) {
      sh.abort_flag = 1;
      if (P.status && lane == 0) atomicOr(P.status, SPECATTN_ROW_TIMEOUT);
    }
  }

  // ---- release tensor memory once every warp that touches it is done -----------------------------
  tc_fence_before();
  named_bar_sync(2, 9 * 32);  // warps 0..8
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
  }
}

template <int NT, bool kPaged>
cudaError_t launch_tc(const VerifyParams& P, const CUtensorMap& kv_map, int n_ctas, cudaStream_t stream) {
  const size_t smem = sizeof(TcShared) + 1024;
  static std::atomic<unsigned long long> done_mask{0};
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!((done_mask.load(std::memory_order_acquire) >> dev) & 1ull)) {
    err = cudaFuncSetAttribute(sparse_verify_tc_kernel<NT, kPaged>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               static_cast<int>(smem));
    if (err != cudaSuccess) return err;
    done_mask.fetch_or(1ull << dev, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(static_cast<unsigned>(n_ctas), 1, 1);
  cfg.blockDim = dim3(kTcThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  err = cudaLaunchKernelEx(&cfg, sparse_verify_tc_kernel<NT, kPaged>, P, kv_map);
  if (err != cudaSuccess) cudaGetLastError();
  return err;
}
