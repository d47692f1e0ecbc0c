// sparse_verify on the 5th-generation tensor cores (tcgen05) -- included by sparse_verify.cu
// inside namespace specattn::{anonymous}; shares VerifyParams, the work partition and the
// cross-CTA merge protocol with the mma.sync kernel there.
//
// Same operation (Eq. 1 over the listed rows, Sec. 3.5 / Alg. 1 "Verification with Sparse
// Attention"), different engine for the two contractions of a 64-key tile:
//   S[128 x 64]  = Q[128 x 128] K^T      one tcgen05.mma chain (8 x K=16), A and B from shared
//                                         memory in the 128-byte-swizzled K-major layout
//   O[128 x 128] += P[128 x 64] V        A = P as packed bf16 in TENSOR MEMORY (two terms,
//                                         P = P_hi + P_lo), B = V from shared memory, MN-major
// The query block ((gamma+1) x group <= 64 rows) sits in rows 0.. of the M = 128 operand, the
// other rows are zero: the tensor pipe has throughput to spare, and in return every query row
// lives in ONE thread of the softmax warps (TMEM lane = row), so max / sum / exp need no
// shuffles and no shared memory at all.
//
// Warp roles (9 warps): 4 producers gather K/V rows with 16-byte cp.async straight into the
// swizzled tile layout (then fence.proxy.async, so the tensor core's async-proxy reads see them);
// 1 warp issues all MMAs and tcgen05.commit arrivals; 2 x 2 softmax warps work on alternate
// tiles, each parity with its own S / P / O columns in TMEM (512 columns in total), and are
// combined at the end of a unit exactly like the key-split warps of the mma.sync kernel.
// The running maximum is only raised when a tile exceeds it by 2^8 (P stays < 256 in bf16);
// raising it rescales the O rows in TMEM (tcgen05.ld / st), which is rare.
#pragma once

constexpr int kTcTile = 64;                      // keys per tile
constexpr int kTcTileBytes = kTcTile * 256;      // one K or V tile (16 KB)
constexpr int kTcRecCols = 130;                  // 128 outputs, m, l of one row
constexpr int kTcRec = kTcRecCols * 32;          // floats of a 32-row record, [column][row]
constexpr float kTcRaise = 8.f;                  // raise the reference maximum beyond 2^8

// byte offset of 16-byte chunk `c` (0..15) of row `r` in a tile of `rows` rows: two 128-byte
// halves per row, chunks XOR-swizzled with the row index (UMMA 128-byte swizzle, K-major)
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
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b), "r"(idesc), "r"(acc), "r"(0u)
      : "memory");
}
// arrival on an mbarrier once every tcgen05 operation issued so far by this thread has completed
__device__ __forceinline__ void tc_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 lanes x 32 columns of 32 bits: thread t of the warp gets / provides TMEM lane (base + t)
#define SPECATTN_TMEM_LD32(r, addr)                                                                             \
  asm volatile(                                                                                                  \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                                  \
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27," \
      "%28,%29,%30,%31}, [%32];"                                                                                 \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),          \
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),    \
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),  \
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])   \
      : "r"(addr))
#define SPECATTN_TMEM_ST32(addr, r)                                                                             \
  asm volatile(                                                                                                  \
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "                                                            \
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28," \
      "%29,%30,%31,%32};" ::"r"(addr),                                                                           \
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),         \
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), \
      "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]),            \
      "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])                                     \
      : "memory")

// NB = 32-row blocks of the query block (1 or 2), NS = ring stages
template <int NB, int NS>
struct TcShared {
  alignas(1024) unsigned char kv[NS][2 * kTcTileBytes];  // per stage: K tile then V tile
  alignas(1024) unsigned char q[128 * 256];
  float scratch[NB][kTcRec];   // parity-1 group -> parity-0 group at the end of a unit
  float peer_rec[NB][kTcRec];  // cluster-pair merge: the odd CTA's records land here
  alignas(8) unsigned long long full[NS];
  unsigned long long empty[NS];
  unsigned long long q_full, q_empty;
  unsigned long long s_full[2], s_free[2], p_full[2], pv_done[2], o_free[2];
  unsigned long long peer_full;
  uint32_t tmem_base;
  int unit_start[kMaxUnits + 1];
  int unit_cnt[kMaxUnits];
  int part_start[kAlignedMaxUnits + 1];
  int cand_parts[kCandidates];
  int cand_max[kCandidates];
  volatile int abort_flag;
};

constexpr int kTcThreads = 9 * 32;
constexpr int kTcMmaWarp = 2;

template <int NB, int NS>
__global__ void __launch_bounds__(kTcThreads, 1) sparse_verify_tc_kernel(const __grid_constant__ VerifyParams P) {
  using Sh = TcShared<NB, NS>;
  extern __shared__ __align__(1024) unsigned char smem_raw_tc[];
  Sh& sh = *reinterpret_cast<Sh*>((reinterpret_cast<uintptr_t>(smem_raw_tc) + 1023) & ~static_cast<uintptr_t>(1023));
  constexpr int NT = kTcThreads;
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const int U = P.B * P.Hkv;

  if (!P.lists_stable) pdl_wait();
  pdl_launch_dependents();

  // ---- set-up ---------------------------------------------------------------------------------
  {
    uint4* zq = reinterpret_cast<uint4*>(sh.q);  // rows beyond the query block stay zero
    for (int i = tid; i < static_cast<int>(sizeof(sh.q) / 16); i += NT) zq[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], 1);
    }
    mbar_init(&sh.q_full, 1);
    mbar_init(&sh.q_empty, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sh.s_full[i], 1);
      mbar_init(&sh.s_free[i], NB);
      mbar_init(&sh.p_full[i], NB);
      mbar_init(&sh.pv_done[i], 1);
      mbar_init(&sh.o_free[i], NB);
    }
    mbar_init(&sh.peer_full, NB);
    mbar_fence_init();
    sh.abort_flag = 0;
    sh.unit_start[0] = 0;
  }
  for (int u = tid; u < U; u += NT) {
    const int c = unit_count(P, u);
    sh.unit_cnt[u] = c;
    sh.unit_start[u + 1] = (c + kAtom - 1) / kAtom;
  }
  fence_proxy_async();
  __syncthreads();
  const bool paired = cluster_num_ctas() == 2;
  if (paired) cluster_sync_all();
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

  // ---- work partition (same two schemes as the mma.sync kernel) ---------------------------------
  const long long N = sh.unit_start[U];
  const int G = static_cast<int>(gridDim.x);
  if (tid < kCandidates) { sh.cand_parts[tid] = 0; sh.cand_max[tid] = 0; }
  __syncthreads();
  const bool try_aligned = (U <= kAlignedMaxUnits) && (N > 0);
  if (try_aligned && tid < U) {
    const int atoms = sh.unit_start[tid + 1] - sh.unit_start[tid];
    if (atoms > 0) {
#pragma unroll
      for (int c = 0; c < kCandidates; ++c) {
        const long long num = static_cast<long long>(atoms) * G * 16;
        const long long den = N * (16 + c);
        int k = static_cast<int>((2 * num + den) / (2 * den));
        if (k < 1) k = 1;
        if (k > atoms) k = atoms;
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
    if (cand >= 0 && static_cast<long long>(sh.cand_max[cand]) * G > N + 24ll * G) cand = -1;
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
          const long long den = N * (16 + cand);
          k = static_cast<int>((2 * num + den) / (2 * den));
          if (k < 1) k = 1;
          if (k > atoms) k = atoms;
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
  const long long NP = aligned ? sh.part_start[U] : ((N < G) ? N : static_cast<long long>(G));

  const bool is_softmax = (warp == 0 || warp == 1 || warp == 4 || warp == 5);
  const bool is_mma = (warp == kTcMmaWarp);
  if (is_softmax || is_mma) {
    // the only warps that write global memory or consume q: the previous kernel is complete
    if (P.lists_stable) pdl_wait();
  }
  if (is_softmax) {
    // units with an empty list: out = 0, lse = -inf
    for (int u = blockIdx.x; u < U; u += gridDim.x) {
      if (sh.unit_cnt[u] != 0) continue;
      const int b = u / P.Hkv, kvh = u % P.Hkv;
      const int st = ((warp & 1) + (warp >> 2) * 2) * 32 + lane;  // 0..127 over the four warps
      for (int e = st; e < P.M * kD; e += 128) {
        const int r = e / kD, t = r / P.grp, h = kvh * P.grp + r % P.grp;
        P.out[((static_cast<long long>(b) * P.T + t) * P.Hq + h) * kD + e % kD] = 0.f;
        if (e % kD == 0) P.lse[(static_cast<long long>(b) * P.T + t) * P.Hq + h] = -INFINITY;
      }
    }
  }
  if (static_cast<long long>(blockIdx.x) >= NP) return;
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
    a0 = cta_first_atom(blockIdx.x, N, NP);
    a1 = cta_first_atom(blockIdx.x + 1, N, NP);
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

  // ---- tensor memory: 512 columns = S[2] (64 each), P_hi[2], P_lo[2] (32 each), O[2] (128 each) --
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;
  auto col_s = [&](int par) { return tmem + static_cast<uint32_t>(par * 64); };
  auto col_phi = [&](int par) { return tmem + 128u + static_cast<uint32_t>(par * 32); };
  auto col_plo = [&](int par) { return tmem + 192u + static_cast<uint32_t>(par * 32); };
  auto col_o = [&](int par) { return tmem + 256u + static_cast<uint32_t>(par * 128); };

  // every role walks the same sequence of segments (unit, token range) and 64-key tiles
  auto next_unit = [&](int& a, int& u, int seg_hi, int ue) {
    a = seg_hi;
    if (a == ue) {
      ++u;
      while (u < U && sh.unit_start[u + 1] == sh.unit_start[u]) ++u;
    }
  };

  if (!is_softmax && !is_mma) {
    // =============================== producer warps ===============================================
    const int pw = (warp == 3) ? 0 : (warp - 5);  // warps 3, 6, 7, 8 -> 0..3
    if (pw < NS) {
      int it = 0, seg = 0;
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
        // the query block of this unit, straight into the swizzled operand layout (warp 0 of
        // the producers only; first segment: after the warp's first tile)
        auto load_q = [&]() -> bool {
          if (seg == 0 && P.lists_stable) pdl_wait();
          if (!mbar_wait(&sh.q_empty, (seg & 1u) ^ 1u, &sh.abort_flag)) return false;
          const uint32_t qb = smem_u32(sh.q);
          for (int i = lane; i < P.M * 16; i += 32) {
            const int r = i >> 4, c = i & 15;
            const int t = r / P.grp, h = kvh * P.grp + r % P.grp;
            cp_async16(qb + tc_sw(r, c, 128), P.q + ((static_cast<long long>(b) * P.T + t) * P.Hq + h) * kD + c * 8);
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
        auto resolve = [&](int t0, long long (&off)[2]) -> bool {
          const int ntok = min(kTcTile, tok_hi - t0);
          bool bad = false;
#pragma unroll
          for (int jj = 0; jj < 2; ++jj) {
            const int jt = min(lane + jj * 32, ntok - 1);
            const int k = t0 + jt;
            int pos = (k >= c_list) ? (kvlen_b + (k - c_list)) : (P.dense ? k : __ldg(list + k));
            if (pos < 0 || pos >= kvlen_b + P.tail) { bad = true; pos = 0; }
            const int lp = (P.page_shift >= 0) ? (pos >> P.page_shift) : (pos / P.page_size);
            const int slot = pos - lp * P.page_size;
            long long page = P.bt ? static_cast<long long>(__ldg(P.bt + b * P.bt_stride + lp))
                                  : (b * P.bt_stride + lp);
            if (page < 0 || (P.n_pages > 0 && page >= P.n_pages)) { bad = true; page = 0; }
            off[jj] = (page * P.s_page + static_cast<long long>(slot) * P.s_slot) * 2;
          }
          return bad;
        };
        long long off_next[2] = {0, 0};
        bool bad_next = false;
        int t0_next = -1;
        for (int t0 = tok_lo; t0 < tok_hi; t0 += kTcTile, ++it) {
          if ((it % NS) != pw) continue;
          const int s = it % NS;
          const unsigned ph = (it / NS) & 1u;
          long long off[2];
          bool bad;
          if (t0_next == t0) {
            off[0] = off_next[0];
            off[1] = off_next[1];
            bad = bad_next;
          } else {
            bad = resolve(t0, off);
          }
          t0_next = t0 + NS * kTcTile;
          if (t0_next < tok_hi) bad_next = resolve(t0_next, off_next); else t0_next = -1;
          if (!mbar_wait(&sh.empty[s], ph ^ 1u, &sh.abort_flag)) { sh.abort_flag = 1; dead = true; break; }
          const int ntok = min(kTcTile, tok_hi - t0);
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
                const uint32_t d = tc_sw(tok, lane & 15, kTcTile);
                cp_async16(k_dst + d, kbase + o);
                cp_async16(v_dst + d, kbase + o + v_delta);
              }
            }
          }
          asm volatile("cp.async.wait_all;" ::: "memory");
          fence_proxy_async();  // generic-proxy writes -> visible to the tensor core's reads
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.full[s]);
          if (bad && P.status) atomicOr(P.status + b, SPECATTN_ROW_BAD_INDEX);
          if (q_pending) {
            q_pending = false;
            if (!load_q()) { sh.abort_flag = 1; dead = true; break; }
          }
        }
        ++seg;
        next_unit(a, u, seg_hi, ue);
      }
    }
    return;
  }

  bool ok = true;
  if (is_mma) {
    // =============================== MMA issue warp (one thread) =================================
    if (lane == 0) {
      const uint32_t idesc_qk = tc_idesc(128, kTcTile, 0, 0);
      const uint32_t idesc_pv = tc_idesc(128, kD, 0, 1);
      const uint32_t q_base = smem_u32(sh.q);
      int it = 0, seg = 0;
      int o_used[2] = {0, 0};  // segments so far in which each parity accumulated
      int a = a0, u = u_first;
      auto issue_pv = [&](int j, int ntok, bool first) {
        const int par = j & 1, s = j % NS;
        const uint32_t v_base = smem_u32(sh.kv[s]) + kTcTileBytes;
        const int ksteps = (ntok + 15) >> 4;
        for (int kk = 0; kk < ksteps; ++kk)
          tc_mma_ts(col_o(par), col_phi(par) + kk * 8, tc_desc(v_base + kk * 2048, 8192, 1024), idesc_pv,
                    (first && kk == 0) ? 0u : 1u);
        for (int kk = 0; kk < ksteps; ++kk)
          tc_mma_ts(col_o(par), col_plo(par) + kk * 8, tc_desc(v_base + kk * 2048, 8192, 1024), idesc_pv, 1u);
        tc_commit(&sh.empty[s]);
        tc_commit(&sh.pv_done[par]);
      };
      while (a < a1 && ok) {
        const int us = sh.unit_start[u], ue = sh.unit_start[u + 1];
        const int seg_hi = min(a1, ue);
        const int tok_lo = (a - us) * kAtom;
        const int tok_hi = min(sh.unit_cnt[u], (seg_hi - us) * kAtom);
        const int ntiles = (tok_hi - tok_lo + kTcTile - 1) / kTcTile;
        if (!mbar_wait(&sh.q_full, seg & 1u, &sh.abort_flag)) { ok = false; break; }
        bool o_waited[2] = {false, false};
        bool first_pv[2] = {true, true};
        for (int n = 0; n <= ntiles && ok; ++n) {
          if (n < ntiles) {  // S = Q K^T of tile it + n
            const int i = it + n, s = i % NS, par = i & 1;
            if (!mbar_wait(&sh.full[s], (i / NS) & 1u, &sh.abort_flag)) { ok = false; break; }
            if (!mbar_wait(&sh.s_free[par], ((i >> 1) & 1u) ^ 1u, &sh.abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t k_base = smem_u32(sh.kv[s]);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              tc_mma_ss(col_s(par), tc_desc(q_base + (kk >> 2) * (128 * 128) + (kk & 3) * 32, 16, 1024),
                        tc_desc(k_base + (kk >> 2) * (kTcTile * 128) + (kk & 3) * 32, 16, 1024), idesc_qk, kk > 0);
            tc_commit(&sh.s_full[par]);
            if (n == ntiles - 1) tc_commit(&sh.q_empty);  // the query tile may be replaced
          }
          if (n > 0) {  // O += P V of tile it + n - 1
            const int j = it + n - 1, par = j & 1;
            if (!o_waited[par]) {  // this parity's O rows of its previous segment have been read out
              if (!mbar_wait(&sh.o_free[par], (o_used[par] & 1u) ^ 1u, &sh.abort_flag)) { ok = false; break; }
              o_waited[par] = true;
            }
            if (!mbar_wait(&sh.p_full[par], (j >> 1) & 1u, &sh.abort_flag)) { ok = false; break; }
            tc_fence_after();
            issue_pv(j, min(kTcTile, tok_hi - (tok_lo + (n - 1) * kTcTile)), first_pv[par]);
            first_pv[par] = false;
          }
        }
        // o_free[par] completes one phase per segment in which that parity had a tile: a parity
        // without one neither arrives nor is waited for, so no phase can ever be skipped
        for (int par = 0; par < 2; ++par)
          if (o_waited[par]) ++o_used[par];
        it += ntiles;
        ++seg;
        next_unit(a, u, seg_hi, ue);
      }
      if (!ok) sh.abort_flag = 1;
    }
    __syncwarp();
  } else {
    // =============================== softmax warps ==============================================
    const int par = warp >> 2;  // tiles with (tile index & 1) == par
    const int rb = warp & 1;    // rows rb * 32 .. rb * 32 + 31 of the query block
    const bool active = rb < NB;
    const int row = rb * 32 + lane;
    const uint32_t lane_sel = static_cast<uint32_t>(rb * 32) << 16;
    const int t_row = row / P.grp;
    const int lim = t_row + P.tail_off;  // last in-flight token this row may see
    int it = 0, seg = 0;
    int a = a0, u = u_first;
    while (active && a < a1) {
      const int us = sh.unit_start[u], ue = sh.unit_start[u + 1];
      const int seg_hi = min(a1, ue);
      const int b = u / P.Hkv, kvh = u % P.Hkv;
      const int tok_lo = (a - us) * kAtom;
      const int tok_hi = min(sh.unit_cnt[u], (seg_hi - us) * kAtom);
      const int c_list = sh.unit_cnt[u] - P.tail;
      const int ntiles = (tok_hi - tok_lo + kTcTile - 1) / kTcTile;
      float m_ref = -INFINITY, l = 0.f;  // reference maximum (scaled log2 domain), row sum
      bool has_acc = false;
      int last_i = -1;
      for (int n = 0; n < ntiles && ok; ++n) {
        const int i = it + n;
        if ((i & 1) != par) continue;
        const int t0 = tok_lo + n * kTcTile;
        const int ntok = min(kTcTile, tok_hi - t0);
        if (!mbar_wait(&sh.s_full[par], (i >> 1) & 1u, &sh.abort_flag)) { ok = false; break; }
        tc_fence_after();
        uint32_t s0[32], s1[32];
        SPECATTN_TMEM_LD32(s0, col_s(par) + lane_sel);
        SPECATTN_TMEM_LD32(s1, col_s(par) + lane_sel + 32);
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.s_free[par]);
        // mask keys that do not exist and in-flight tokens this row may not see yet
        const int tb = P.tail ? (c_list - t0) : (1 << 20);
        float tmax = -INFINITY;
#pragma unroll
        for (int k = 0; k < 32; ++k) {
          float x = __uint_as_float(s0[k]), y = __uint_as_float(s1[k]);
          if (k >= ntok || (k - tb >= 0 && k - tb > lim)) x = -INFINITY;
          if (k + 32 >= ntok || (k + 32 - tb >= 0 && k + 32 - tb > lim)) y = -INFINITY;
          s0[k] = __float_as_uint(x);
          s1[k] = __float_as_uint(y);
          tmax = fmaxf(tmax, fmaxf(x, y));
        }
        tmax *= P.scale_log2;
        // P[par] and O[par] are quiet once the P V product of this parity's previous tile is done
        if (!mbar_wait(&sh.pv_done[par], ((i >> 1) & 1u) ^ 1u, &sh.abort_flag)) { ok = false; break; }
        tc_fence_after();
        const bool raise = (tmax > m_ref + kTcRaise) || (m_ref == -INFINITY && tmax > -INFINITY);
        if (__any_sync(0xffffffffu, raise && has_acc)) {
          // rescale this warp's O rows in tensor memory (rows that do not raise scale by 1)
          const float alpha = (raise && has_acc) ? ex2(m_ref - tmax) : 1.f;
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t o[32];
            SPECATTN_TMEM_LD32(o, col_o(par) + lane_sel + c * 32);
            tc_wait_ld();
#pragma unroll
            for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
            SPECATTN_TMEM_ST32(col_o(par) + lane_sel + c * 32, o);
          }
          tc_wait_st();
        }
        if (raise) {
          l *= (m_ref == -INFINITY) ? 0.f : ex2(m_ref - tmax);
          m_ref = tmax;
        }
        const float base = (m_ref == -INFINITY) ? 0.f : m_ref;
        float sum = 0.f;
        uint32_t phi[32], plo[32];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const float x0 = ex2(fmaf(__uint_as_float(s0[2 * k]), P.scale_log2, -base));
          const float x1 = ex2(fmaf(__uint_as_float(s0[2 * k + 1]), P.scale_log2, -base));
          const float y0 = ex2(fmaf(__uint_as_float(s1[2 * k]), P.scale_log2, -base));
          const float y1 = ex2(fmaf(__uint_as_float(s1[2 * k + 1]), P.scale_log2, -base));
          sum += (x0 + x1) + (y0 + y1);
          const uint32_t hx = pack_bf16(x0, x1), hy = pack_bf16(y0, y1);
          phi[k] = hx;
          phi[16 + k] = hy;
          plo[k] = pack_bf16(x0 - __uint_as_float(hx << 16), x1 - __uint_as_float(hx & 0xffff0000u));
          plo[16 + k] = pack_bf16(y0 - __uint_as_float(hy << 16), y1 - __uint_as_float(hy & 0xffff0000u));
        }
        l += sum;
        SPECATTN_TMEM_ST32(col_phi(par) + lane_sel, phi);
        SPECATTN_TMEM_ST32(col_plo(par) + lane_sel, plo);
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.p_full[par]);
        has_acc = true;
        last_i = i;
      }
      // ---- end of the unit's share: read this parity's O rows, hand the columns back -----------
      float acc[kD];
      if (ok && has_acc) {
        if (!mbar_wait(&sh.pv_done[par], (last_i >> 1) & 1u, &sh.abort_flag)) ok = false;
        tc_fence_after();
      }
      if (ok && has_acc) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t o[32];
          SPECATTN_TMEM_LD32(o, col_o(par) + lane_sel + c * 32);
          tc_wait_ld();
#pragma unroll
          for (int k = 0; k < 32; ++k) acc[c * 32 + k] = __uint_as_float(o[k]);
        }
      } else {
#pragma unroll
        for (int k = 0; k < kD; ++k) acc[k] = 0.f;
      }
      tc_fence_before();
      __syncwarp();
      if (has_acc && lane == 0) mbar_arrive(&sh.o_free[par]);
      if (!ok) sh.abort_flag = 1;

      // combine the two parities of this row block (warps w and w + 4) through shared memory
      float m = m_ref;
      if (par == 1) {
        float* rec = sh.scratch[rb];
#pragma unroll
        for (int k = 0; k < kD; ++k) rec[k * 32 + lane] = acc[k];
        rec[128 * 32 + lane] = m;
        rec[129 * 32 + lane] = l;
      }
      named_bar_sync(1 + rb, 64);
      if (par == 0) {
        const float* rec = sh.scratch[rb];
        float mn, ao, ai;
        merge_scales(m, rec[128 * 32 + lane], mn, ao, ai);
        l = l * ao + rec[129 * 32 + lane] * ai;
        m = mn;
#pragma unroll
        for (int k = 0; k < kD; ++k) acc[k] = acc[k] * ao + rec[k * 32 + lane] * ai;
      }
      named_bar_sync(1 + rb, 64);
      if (sh.abort_flag) { ok = false; break; }

      if (par == 0) {
        const bool whole = (a == us) && (seg_hi == ue);
        bool finish = whole;
        const bool pair_merge = paired && aligned && !whole && (sh.part_start[u + 1] - sh.part_start[u] == 2) &&
                                ((sh.part_start[u] & 1) == 0);
        if (pair_merge) {
          if (cluster_cta_rank() == 1) {
            const uint32_t dst = map_to_cta(smem_u32(sh.peer_rec[rb]), 0) + lane * 4;
#pragma unroll
            for (int k = 0; k < kD; ++k) st_cluster_f32(dst + k * 128, acc[k]);
            st_cluster_f32(dst + 128 * 128, m);
            st_cluster_f32(dst + 129 * 128, l);
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(map_to_cta(smem_u32(&sh.peer_full), 0));
          } else {
            if (!mbar_wait_cluster(&sh.peer_full, 0u, &sh.abort_flag)) { sh.abort_flag = 1; ok = false; break; }
            const float* rec = sh.peer_rec[rb];
            float mn, ao, ai;
            merge_scales(m, rec[128 * 32 + lane], mn, ao, ai);
            l = l * ao + rec[129 * 32 + lane] * ai;
            m = mn;
#pragma unroll
            for (int k = 0; k < kD; ++k) acc[k] = acc[k] * ao + rec[k * 32 + lane] * ai;
            finish = true;
          }
        } else if (!whole) {
          float* rec = P.partials + (static_cast<size_t>(2 * blockIdx.x + (a == a0 ? 0 : 1)) * NB + rb) * kTcRec;
#pragma unroll
          for (int k = 0; k < kD; ++k) __stcg(rec + k * 32 + lane, acc[k]);
          __stcg(rec + 128 * 32 + lane, m);
          __stcg(rec + 129 * 32 + lane, l);
          __threadfence();
          __syncwarp();
          const int i_lo = aligned ? sh.part_start[u] : cta_of_atom(us, N, NP);
          const int i_hi = aligned ? sh.part_start[u + 1] - 1 : cta_of_atom(ue - 1, N, NP);
          unsigned int old = 0;
          if (lane == 0) old = atomicAdd(P.counters + u * kCountersPerUnit + rb, 1u);
          old = __shfl_sync(0xffffffffu, old, 0);
          if (old == static_cast<unsigned int>(i_hi - i_lo)) {
            finish = true;
            __threadfence();
            // merge every contributor's record in CTA order (the own one included, from memory)
            m = -INFINITY;
            for (int i = i_lo; i <= i_hi; ++i) {
              const float* r2 = P.partials +
                  (static_cast<size_t>(2 * i + ((aligned || cta_first_atom(i, N, NP) >= us) ? 0 : 1)) * NB + rb) * kTcRec;
              m = fmaxf(m, __ldcg(r2 + 128 * 32 + lane));
            }
            const float base = (m == -INFINITY) ? 0.f : m;
            l = 0.f;
#pragma unroll
            for (int k = 0; k < kD; ++k) acc[k] = 0.f;
            for (int i = i_lo; i <= i_hi; ++i) {
              const float* r2 = P.partials +
                  (static_cast<size_t>(2 * i + ((aligned || cta_first_atom(i, N, NP) >= us) ? 0 : 1)) * NB + rb) * kTcRec;
              const float w = ex2(__ldcg(r2 + 128 * 32 + lane) - base);
              l += __ldcg(r2 + 129 * 32 + lane) * w;
#pragma unroll
              for (int k = 0; k < kD; ++k) acc[k] += __ldcg(r2 + k * 32 + lane) * w;
            }
            if (lane == 0) P.counters[u * kCountersPerUnit + rb] = 0u;
          }
        }
        if (finish && row < P.M) {
          const float inv = (l > 0.f) ? 1.f / l : 0.f;
          const int h = kvh * P.grp + row % P.grp;
          const long long orow = (static_cast<long long>(b) * P.T + t_row) * P.Hq + h;
          float4* o = reinterpret_cast<float4*>(P.out + orow * kD);
#pragma unroll
          for (int k = 0; k < kD / 4; ++k)
            o[k] = make_float4(acc[4 * k] * inv, acc[4 * k + 1] * inv, acc[4 * k + 2] * inv, acc[4 * k + 3] * inv);
          P.lse[orow] = (l > 0.f) ? (m + log2f(l)) * kLn2 : -INFINITY;
        }
      }
      it += ntiles;
      ++seg;
      next_unit(a, u, seg_hi, ue);
    }
    if (!ok && P.status && lane == 0) atomicOr(P.status, SPECATTN_ROW_TIMEOUT);
  }

  // ---- release tensor memory once every warp that touches it is done -----------------------------
  tc_fence_before();
  named_bar_sync(5, 5 * 32);  // warps 0, 1, 2, 4, 5
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

template <int NB, int NS>
cudaError_t launch_tc(const VerifyParams& P, int n_ctas, cudaStream_t stream) {
  const size_t smem = sizeof(TcShared<NB, NS>) + 1024;
  static std::atomic<unsigned long long> done_mask{0};
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!((done_mask.load(std::memory_order_acquire) >> dev) & 1ull)) {
    err = cudaFuncSetAttribute(sparse_verify_tc_kernel<NB, NS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
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
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (n_ctas % 2 == 0) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  err = cudaLaunchKernelEx(&cfg, sparse_verify_tc_kernel<NB, NS>, P);
  if (err != cudaSuccess) cudaGetLastError();
  return err;
}
