/* specattn.h -- C ABI of the SpecAttn verification hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, as hand-written CUDA kernels, the per-step work that the SpecAttn
 * verifier performs for each of its layers:
 *
 *   select:  sum the mapped draft layer's attention probabilities over draft heads and the
 *            gamma speculated queries, find the exact top-p nucleus of context positions
 *            without sorting (a radix threshold search over the binary32 bit pattern with
 *            per-bin counts and masses) and emit the kept positions as ascending index lists.
 *   verify:  grouped-query sparse decode attention of the gamma+1 verification queries over
 *            only the listed rows of a paged bf16 K/V cache, returning outputs and LSE.
 *
 * Conventions common to every entry point
 *   - Pointers are DEVICE pointers unless the comment says HOST.  The caller owns every
 *     buffer; the library never allocates or frees device memory and never synchronises.
 *     Work is enqueued on the CUDA stream passed as `cuda_stream` (a cudaStream_t cast to
 *     void*; NULL = the legacy default stream) and is complete when that stream reaches it.
 *   - Return value: SPECATTN_OK (0) = enqueued; a negative SPECATTN_ERR_* = argument error
 *     detected on the host, nothing was launched.  Data-dependent problems are reported per
 *     list / per sequence in device status words as SPECATTN_ROW_* bit flags; the device
 *     code never traps.
 *   - `struct_size` must be sizeof() of the struct the caller was compiled against.
 *   - Strides are in ELEMENTS of the array they index.
 *   - Tracing: specattn_select_topp, specattn_sparse_verify, specattn_verify_plan(_many) and
 *     specattn_verify_step_host each open an NVTX range of their own name around their host-side
 *     work (visible in a profiler's timeline; a null-pointer test when no tool is attached).
 */
#ifndef SPECATTN_H_
#define SPECATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- host-side return codes ------------------------------------------------------------ */
#define SPECATTN_OK 0
#define SPECATTN_ERR_NULL (-1)        /* a required pointer is NULL */
#define SPECATTN_ERR_STRUCT_SIZE (-2) /* struct_size does not match this library */
#define SPECATTN_ERR_RANGE (-3)       /* a scalar is outside its documented range */
#define SPECATTN_ERR_ALIGN (-4)       /* a pointer or stride breaks the 16-byte rules */
#define SPECATTN_ERR_WORKSPACE (-5)   /* workspace missing or smaller than *_workspace_bytes() */
#define SPECATTN_ERR_UNSUPPORTED (-6) /* shape outside what the kernels are built for */
#define SPECATTN_ERR_CUDA (-7)        /* the CUDA runtime refused the launch */
#define SPECATTN_ERR_STATIC_SCRATCH (-8) /* shape needs more scratch than the built-in buffer has */

/* ---- device-side per-list / per-sequence status flags ---------------------------------- */
#define SPECATTN_ROW_OK 0
#define SPECATTN_ROW_INVALID_PROB 1 /* a contributing probability was negative, NaN or Inf (or the
                                       binary32 sum of a position overflowed) */
#define SPECATTN_ROW_OVERFLOW 2     /* the list has more entries than idx_stride; truncated */
#define SPECATTN_ROW_BAD_INDEX 4    /* verify met a position or page id out of range */
#define SPECATTN_ROW_TIMEOUT 8      /* a bounded device-side wait ran out; outputs invalid */

/* ---- limits ---------------------------------------------------------------------------- */
#define SPECATTN_MAX_DRAFT_LAYERS 64
#define SPECATTN_MAX_DRAFT_HEADS 256
#define SPECATTN_MAX_ROWS_PER_LIST 1024  /* contributing (head, query) rows per list */
#define SPECATTN_MAX_KV_LEN 196608       /* positions per sequence for select (8 x 24576) */
#define SPECATTN_MAX_VERIFY_UNITS 2048   /* batch * n_kv_heads for verify */
#define SPECATTN_MAX_QUERY_ROWS 64       /* n_q * (n_q_heads / n_kv_heads) for verify */

/* ========================================================================================
 * specattn_select_topp -- token selection.
 *
 * Paper: Sec. 3.4 ("Sorting-Free Top-p Nucleus Selection"), Alg. 2, and the top-p objective
 * of App. A Eq. 7; the per-layer use is Alg. 1, block "Sparse Attention Mask Creation".
 *
 * For every draft layer u that some target layer maps to (layer_map[j] == u), every sequence
 * b and every group g:
 *   a_bar[i] = +0 + sum over heads h feeding g (ascending) of sum over s < gamma (ascending)
 *              of draft_probs[u][b, h, s, i],   i < kv_len[b]        (binary32 adds, this order)
 *   total    = sum_i a_bar[i];  target = (double) p * total            (Alg. 2: p * sum a)
 *   theta    = the largest row value v whose mass {a_bar >= v} reaches target -- the fixed
 *              point of Alg. 2's bisection, identical to the sorted-prefix nucleus of Eq. 7
 *   list     = ascending { i : a_bar[i] >= theta }  (ties at theta all kept)
 *   p >= 1 keeps every position; an all-zero row keeps every position.
 * Draft layers no target layer maps to are skipped and their outputs left untouched.
 *
 * Outputs per (u, b, g), all indexed [n_draft_layers, batch, n_groups]:
 *   idx     int32 [.., idx_stride]: the list, first min(count, idx_stride) entries
 *   counts  int32: the true list length (also when it exceeds idx_stride)
 *   row_status int32: SPECATTN_ROW_* flags.  INVALID_PROB => count 0, list unspecified.
 *   diag    optional double [.., 4] = {total, target, mass strictly above theta,
 *           mass of the kept set}; NULL to skip.
 *
 * Variants of Alg. 2 (both off by default; results differ from the exact nucleus by design):
 *   per_step = 1: Alg. 2 as printed -- every speculated query s gets its own row
 *       a_s[i] = +0 + sum over heads h feeding g (ascending) of draft_probs[u][b, h, s, i], its
 *       own threshold, and the list is the ascending union of the gamma sets.
 *   bisect_iters = n in [1, 64]: the threshold of a row is the LAST midpoint of n bisection
 *       steps (theta_high = max of the row, theta_low = 0, theta_mid = (high + low) / 2 in
 *       binary32; mass of {a >= theta_mid} < target lowers theta_high, otherwise raises
 *       theta_low) -- the paper's implementation uses n = 10.  The set {a >= theta_mid} may fall
 *       short of the target mass or exceed the smallest set.  p >= 1 and all-zero rows still
 *       keep every position.  diag then describes the exact threshold of the last row searched.
 *
 *   chunk = c in {4, 8, 16, 32, 64} (0 or 1 = off): selection at chunk granularity (Sec. 4 sets
 *       the chunk size to 16; how a chunk is scored is not stated -- here: its score is
 *       +0 + a[c j] + a[c j + 1] + ... in binary32, ascending, the last chunk cut at kv_len).  The
 *       nucleus (either variant above applies) is taken over the row of chunk scores and a kept
 *       chunk keeps all its positions; counts / idx_stride stay in positions.
 *
 * Requirements: 1 <= n_draft_layers <= 64; n_draft_heads <= 256; gamma >= 1; L_stride a
 * multiple of 4 and <= SPECATTN_MAX_KV_LEN; every draft_probs[u] 16-byte aligned;
 * 0 <= kv_len[b] <= L_stride (larger values are clamped); 0 < p (NaN rejected);
 * n_groups >= 1; head_group (HOST, may be NULL = every head feeds every group) values in
 * [0, n_groups).
 *
 * workspace (optional, device, 16-byte aligned, specattn_select_workspace_bytes() bytes; no
 * counterpart in the paper): without it each list is aggregated and searched inside the shared
 * memory of one thread-block cluster (at most 8 CTAs per list, one launch).  With it, and for
 * the default selection (no variant) over rows of >= 2048 positions when the lists are so few
 * that one cluster each would leave SMs idle (lists x CTAs per cluster < 148), the call runs two
 * launches: every list's rows are summed by CTAs of 512 positions each -- in the same order,
 * so a[] has the same bits -- into the workspace, and the search then reads a[] from there; the
 * lists are the same, the GPU is filled whatever the number of lists.  The workspace holds no
 * state between calls; two calls that may overlap on the GPU need separate workspaces.
 *
 * form: which of the two the call takes when both apply (a workspace is given, default selection,
 * multi-row lists of >= 2048 positions).  SPECATTN_SELECT_FORM_AUTO decides by what the host
 * can see (the number of lists).  What it cannot see is kv_len: in a ragged batch one cluster per
 * list means the longest list sets the time while most of the GPU is done, and the two-launch
 * form, whose first launch spends CTAs in proportion to each list's length, is the better one --
 * a caller that knows its batch is ragged says SPECATTN_SELECT_FORM_TWO_LAUNCH
 * (specattn_select_workspace_bytes then answers for that form).  SPECATTN_SELECT_FORM_CLUSTER
 * keeps one launch.  The lists are the same bits in every form.
 * ======================================================================================== */
#define SPECATTN_SELECT_FORM_AUTO 0
#define SPECATTN_SELECT_FORM_CLUSTER 1
#define SPECATTN_SELECT_FORM_TWO_LAUNCH 2

typedef struct specattn_select_args {
  uint32_t struct_size;
  int32_t n_draft_layers;
  int32_t n_target_layers;
  int32_t batch;
  int32_t n_draft_heads;
  int32_t gamma;
  int32_t n_groups;
  int64_t L_stride;
  const float* const* draft_probs; /* HOST array [n_draft_layers] of device pointers to
                                      binary32 [batch, n_draft_heads, gamma, L_stride];
                                      entries of unmapped layers may be NULL */
  const int32_t* kv_len;           /* [batch] */
  const int32_t* layer_map;        /* HOST [n_target_layers], values in [-1, n_draft_layers);
                                      -1 marks a dense target layer */
  const int32_t* head_group;       /* HOST [n_draft_heads] or NULL */
  float p;
  int32_t* idx;
  int64_t idx_stride;
  int32_t* counts;
  int32_t* row_status;
  double* diag;
  int32_t per_step;     /* 0 | 1 */
  int32_t bisect_iters; /* 0 = exact threshold, else 1..64 */
  int32_t chunk;        /* 0 | 1 = per position, else 4, 8, 16, 32 or 64 */
  int32_t form;         /* SPECATTN_SELECT_FORM_*: 0 = the library picks */
  void* workspace;          /* device, or NULL */
  uint64_t workspace_bytes; /* size of *workspace */
} specattn_select_args;

int specattn_select_topp(const specattn_select_args* args, void* cuda_stream);

/* Bytes of workspace that let specattn_select_topp(args) take its two-launch form (0 when the
 * call would not use one: a variant, single-row lists, rows shorter than 2048 positions, enough
 * lists to fill the GPU with one cluster each, or invalid arguments).  Reads only the scalar fields and layer_map of args. */
size_t specattn_select_workspace_bytes(const specattn_select_args* args);

/* ========================================================================================
 * specattn_sparse_verify -- sparse attention of one target layer.
 *
 * Paper: Eq. 1 restricted to the selected index set I of Eq. 2-3 (softmax normalised over I;
 * the un-normalised form of Eq. 2 is out * exp(lse - lse_dense)); Sec. 3.5; Alg. 1, block
 * "Verification with Sparse Attention" (one list per layer shared by all gamma+1 queries).
 *
 * For sequence b, query t < n_q and query head h (kv head hk = h / (n_q_heads/n_kv_heads),
 * list g = 0 if n_groups == 1 else hk):
 *   s_i = sm_scale * q[b,t,h,:] . K[i, hk, :]  for i in the list;  m = max s_i
 *   out[b,t,h,:] = sum_i exp(s_i - m) V[i, hk, :] / sum_i exp(s_i - m)
 *   lse[b,t,h]   = m + ln sum_i exp(s_i - m)          (natural log)
 * An empty list gives out = 0, lse = -inf.  Position i of sequence b lives in page
 * block_table[b * block_table_stride + i / page_size] at slot i % page_size; with
 * block_table == NULL the cache is contiguous and that page is
 * b * block_table_stride + i / page_size (block_table_stride = pages per sequence).
 * Element (page, kv, slot, head, e) of kv_pages is at
 *   page*stride_page + kv*stride_kv + slot*stride_slot + head*stride_head + e,
 * kv = 0 for keys and 1 for values.
 *
 * idx / counts point at the lists of ONE draft layer: idx [batch, n_groups, idx_stride],
 * counts [batch, n_groups] (entries beyond idx_stride are ignored).  dense != 0 attends every
 * position below kv_len[b] and reads neither idx nor counts (both may be NULL).
 *
 * tail_len > 0 adds the tokens being verified themselves (Alg. 1: the gamma+1 tokens go through
 * the verifier in one pass): their K/V rows must already be in the cache at positions
 * kv_len[b] + j, j < tail_len, and query t attends, after its list, the rows with
 * j <= t + (tail_len - n_q) -- with tail_len == n_q token t sees tokens 0..t.  kv_len stays the
 * context length without them.
 *
 * Requirements: head_dim == 128; n_q * (n_q_heads / n_kv_heads) <= 64; batch * n_kv_heads
 * <= 2048; q, kv_pages 16-byte aligned and all four strides multiples of 8; out 16-byte
 * aligned.  status (int32 [batch], optional) receives SPECATTN_ROW_BAD_INDEX when a listed
 * position is outside [0, kv_len[b]) or a page id outside [0, n_pages) (such entries are
 * read from position 0 / page 0 instead; n_pages == 0 disables the page check).
 *
 * workspace: at least specattn_verify_workspace_bytes() bytes, 256-byte aligned, prepared
 * once with specattn_verify_workspace_init() and then reusable by consecutive calls on the
 * same stream; two calls that may overlap on the GPU need separate workspaces.
 * ======================================================================================== */
/* flags for specattn_verify_args.flags
 *
 * SPECATTN_VERIFY_LISTS_STABLE: the caller promises that idx, counts, kv_len, block_table and
 * the listed rows of kv_pages were produced at least two launches earlier in the stream, and
 * that the launch right before this call is either another specattn_sparse_verify call or a
 * kernel that does not signal programmatic launch completion early.  (True for every layer
 * after the first of a step: the lists come from specattn_select_topp and the context's K/V
 * rows are old.)  The verify kernel is always launched with programmatic stream
 * serialization, i.e. it may begin while the preceding kernel is still running.  Without this
 * flag it waits for that kernel to finish before reading anything, and lets its own successor
 * start only after that wait; with it, it starts fetching K/V rows at once and waits only
 * before reading q and before writing out, lse, status or the workspace.
 *
 * SPECATTN_VERIFY_ENGINE_MMA_SYNC / SPECATTN_VERIFY_ENGINE_TCGEN05: force one of the two
 * implementations of the same operation (warp-level mma.sync with register accumulators, or
 * tcgen05.mma with accumulators in tensor memory).  With neither bit the library picks by
 * what the host can see: tcgen05 for dense calls over caches of at least 8192 positions per
 * sequence (block_table_stride * page_size) that either have more than 32 query rows per KV head
 * (n_q * n_q_heads / n_kv_heads) or can be read page-wise (page_size a multiple of 16, n_pages
 * given), mma.sync otherwise -- list lengths live on the device, so a
 * caller that knows its lists are long (thousands of positions per sequence) and has more than
 * 32 query rows should set SPECATTN_VERIFY_ENGINE_TCGEN05 itself.  Results agree within the
 * tolerance of the operation either way.  Setting both bits is SPECATTN_ERR_RANGE. */
#define SPECATTN_VERIFY_LISTS_STABLE 1u
#define SPECATTN_VERIFY_ENGINE_MMA_SYNC 2u
#define SPECATTN_VERIFY_ENGINE_TCGEN05 4u
/* SPECATTN_VERIFY_PAGE_LISTS: the caller promises that every list consists of whole aligned
 * 16-position chunks -- entries 16 a ... 16 a + 15 are 16 consecutive positions starting at a
 * multiple of 16, for every a; only the last chunk of a list may be shorter (cut at kv_len or at
 * idx_stride).  Lists written by specattn_select_topp with chunk = 16, 32 or 64 have this form
 * (Sec. 4: chunk size 16).  Where the cache's page size is a multiple of 16 and n_pages is given,
 * the kernel then reads K/V page-wise -- one list entry, one block-table entry and four tiled
 * bulk tensor copies (16 slots x 128 bytes each) per 16 tokens instead of 16 entries and 512
 * 16-byte copies -- and so does every dense call.  A list that breaks the promise gives wrong
 * results for its sequence (entries that are not multiples of 16 raise SPECATTN_ROW_BAD_INDEX),
 * never a fault.  Results are the same as without the flag. */
#define SPECATTN_VERIFY_PAGE_LISTS 8u
/* TEST ONLY -- never set this in production.  Exercises the failure path of the kernels' bounded
 * device-side waits without faulting anything: one producer warp of CTA 0 withholds the
 * completion signal of its first tile, the waits on it give up after their poll limit (about
 * half a second each), the CTA raises SPECATTN_ROW_TIMEOUT in status[0] and the kernel returns
 * normally.  Outputs of that call are invalid and the workspace must be re-initialised with
 * specattn_verify_workspace_init before its next use. */
#define SPECATTN_VERIFY_TEST_LOSE_ARRIVAL 0x80000000u

typedef struct specattn_verify_args {
  uint32_t struct_size;
  int32_t batch;
  int32_t n_q;
  int32_t n_q_heads;
  int32_t n_kv_heads;
  int32_t head_dim;
  int32_t page_size;
  int32_t n_groups;
  int32_t dense;
  const void* q;        /* bf16 [batch, n_q, n_q_heads, head_dim] */
  const void* kv_pages; /* bf16 pool of this target layer */
  int64_t n_pages;
  int64_t stride_page, stride_kv, stride_slot, stride_head;
  const int32_t* block_table;
  int64_t block_table_stride;
  const int32_t* kv_len; /* [batch] */
  const int32_t* idx;
  int64_t idx_stride;
  const int32_t* counts;
  float sm_scale;        /* > 0, or 0 => 1/sqrt(head_dim); negative or NaN is rejected */
  float* out;            /* binary32 [batch, n_q, n_q_heads, head_dim] */
  float* lse;            /* binary32 [batch, n_q, n_q_heads] */
  int32_t* status;       /* [batch] or NULL */
  void* workspace;
  size_t workspace_bytes;
  uint32_t flags;        /* SPECATTN_VERIFY_* bits, 0 for none */
  int32_t tail_len;      /* in-flight tokens attended causally after the list, 0 <= tail_len <= 64 */
  const void* plan;      /* optional: a work partition made by specattn_verify_plan, or NULL */
} specattn_verify_args;

/* Bytes of workspace specattn_sparse_verify needs for these shapes on the current device
 * (0 on argument error).  Depends only on the scalar fields. */
size_t specattn_verify_workspace_bytes(const specattn_verify_args* args);

/* Zero the arrival counters at the head of a verify workspace (enqueued on the stream).
 * Call once after allocating it; the kernels leave the counters zero when they finish. */
int specattn_verify_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream);

int specattn_sparse_verify(const specattn_verify_args* args, void* cuda_stream);

/* specattn_verify_plan -- the work partition of a verify launch, computed ahead of it.
 *
 * Not an operation of the paper: an engineering shortcut of this implementation.  How the kernel
 * deals its (sequence, kv head) lists to the SMs depends only on the list lengths (counts, or
 * kv_len for dense calls), tail_len, the shapes and the GPU -- not on q, the K/V pool or the
 * outputs.  Target layers that share a draft layer's lists therefore share the partition, and a
 * verify kernel that finds a matching plan in args->plan skips computing it (a few microseconds
 * of start-up per launch).  `plan` is a device buffer of specattn_verify_plan_bytes(args) bytes,
 * 16-byte aligned, written by a small kernel on the stream (after whatever produces counts /
 * kv_len, e.g. specattn_select_topp) and valid until those change.  A kernel given a plan that
 * does not fit its launch (other batch, heads, tail_len, dense flag or GPU) ignores it.  Only
 * the mma.sync engine reads plans.
 * Ordering: a plan must be at least as new as the lists it describes -- call this after every
 * specattn_select_topp that rewrites counts -- and a verify call flagged
 * SPECATTN_VERIFY_LISTS_STABLE must not be the first launch after the plan kernel (that flag's
 * "two launches earlier" rule covers the plan like the lists): the plan kernel signals completion
 * only when it has finished, and the first verify call after it waits for that. */
size_t specattn_verify_plan_bytes(const specattn_verify_args* args);
int specattn_verify_plan(const specattn_verify_args* args, void* plan, size_t plan_bytes, void* cuda_stream);
/* The same for n launches at once (HOST arrays of n argument structs, plan buffers and their
 * sizes): one kernel launch per eight plans instead of one per plan -- a step whose target
 * layers share the lists of four draft layers needs four plans. */
int specattn_verify_plan_many(const specattn_verify_args* const* args, void* const* plans,
                              const size_t* plan_bytes, int32_t n, void* cuda_stream);

/* ========================================================================================
 * specattn_sparse_verify_static -- specattn_sparse_verify for callers that cannot allocate.
 *
 * (No counterpart in the paper: this entry point exists only for integration.)
 *
 * Some callers have no way to obtain the scratch buffer specattn_sparse_verify wants: code
 * running as a custom call inside another runtime's compiled graph is handed its input and
 * output buffers and nothing else; a serving engine may have reserved all device memory in
 * its own pool, so that a cudaMalloc from a plug-in fails or stalls the whole device; and
 * an allocation in the middle of a latency-critical decode loop synchronises the GPU.
 * For them this variant keeps the scratch inside the library: a file-scope
 * `static __device__` array of SPECATTN_STATIC_SCRATCH_BYTES bytes that every GPU loading the
 * library holds from load until the process exits.  The call allocates and frees nothing
 * (no cudaMalloc, cudaFree or allocating library routine).
 *
 * Same arguments, results and status codes as specattn_sparse_verify, except:
 *   - args->workspace and args->workspace_bytes are ignored;
 *   - a shape whose scratch need (specattn_verify_workspace_bytes) exceeds
 *     SPECATTN_STATIC_SCRATCH_BYTES is rejected with SPECATTN_ERR_STATIC_SCRATCH and nothing
 *     is launched.  The buffer covers up to 32 query rows per KV head (n_q * group <= 32) on
 *     GPUs with up to 160 SMs;
 *   - the first call on each device looks up the device address of the array (with that
 *     device current); make that first call outside any stream capture;
 *   - all calls on a device share the one array, which still holds what the previous call left
 *     there: the arrival counters are cleared on the stream at the start of every call, and
 *     two calls that may overlap on the GPU (different streams, or concurrent graph branches)
 *     race on it -- serialise them or use specattn_sparse_verify with separate workspaces;
 *   - the clearing is a memset in front of the launch, so a call flagged
 *     SPECATTN_VERIFY_LISTS_STABLE gains nothing here: the kernel cannot begin under its
 *     predecessor as it does after specattn_sparse_verify, it starts when the memset is done;
 *   - every argument check happens before the memset is enqueued: a negative return code means
 *     that nothing at all was enqueued.
 * ======================================================================================== */
#define SPECATTN_STATIC_SCRATCH_BYTES (6u << 20)

int specattn_sparse_verify_static(const specattn_verify_args* args, void* cuda_stream);

/* ========================================================================================
 * specattn_verify_step_host -- one whole verification step from HOST buffers.
 *
 * Alg. 1, blocks "Sparse Attention Mask Creation" and "Verification with Sparse Attention":
 * one select over the mapped draft layers, then one sparse verify per target layer, with the
 * step's inputs and results crossing PCIe inside the call.  It
 *   1. copies q_host[j] -> verify[j].q for every target layer and draft_probs_host[u] ->
 *      select.draft_probs[u] for every mapped draft layer, on a copy stream of its own,
 *   2. on the caller's stream runs specattn_select_topp for a draft layer as soon as its rows
 *      have landed (one launch per mapped draft layer) and then specattn_sparse_verify(verify[j])
 *      of the target layers mapped to it, while later draft layers are still being copied,
 *   3. copies verify[j].out / .lse -> out_host[j] / lse_host[j] on a second copy stream as each
 *      layer finishes,
 * and finally makes the caller's stream wait for both copy streams: work enqueued on that
 * stream afterwards sees the step complete.  The two copy streams and the events between the
 * lanes are created on the first call per device and kept; one call at a time enqueues per
 * device.  select.n_target_layers must equal n_target_layers.  Where verify[j].plan is set, the
 * call runs specattn_verify_plan into it before the first layer that points at it.
 * `select` and `verify[j]` are complete device-side argument structs (their device buffers,
 * including the staging buffers the copies land in, are the caller's); verify[j].idx/counts
 * must already point at the lists of layer_map[j] (or dense be set where layer_map[j] < 0).
 * Host buffers should be pinned for the copies to be asynchronous.  Nothing is synchronised:
 * the results are in the host buffers once the stream has drained.
 * ======================================================================================== */
typedef struct specattn_step_host_args {
  uint32_t struct_size;
  int32_t n_target_layers;
  const specattn_select_args* select;     /* HOST */
  const float* const* draft_probs_host;   /* HOST [n_draft_layers] of HOST pointers */
  const specattn_verify_args* verify;     /* HOST [n_target_layers] */
  const void* const* q_host;              /* HOST [n_target_layers] of HOST pointers (bf16) */
  float* const* out_host;                 /* HOST [n_target_layers] of HOST pointers */
  float* const* lse_host;                 /* HOST [n_target_layers] of HOST pointers */
} specattn_step_host_args;

int specattn_verify_step_host(const specattn_step_host_args* args, void* cuda_stream);

/* Text for a SPECATTN_ERR_* return code (static storage, never NULL). */
const char* specattn_status_string(int code);

/* Number of kernels this library has launched in the calling process since load (for
 * accounting in benchmarks); thread-safe. */
int64_t specattn_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SPECATTN_H_ */
