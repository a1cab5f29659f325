/*
 * nsp.h -- C ABI of the B200 (sm_100a) library for the local attention compute phase of nested sequence
 * parallelism: packed variable-length causal GQA attention, forward and backward, over ONE GPU's share of a
 * nested plan.
 *
 * Where the operation comes from (paper sections):
 *   - Sec. 2.1, paragraph "Sequence Parallelism": after the Ulysses all-to-all a GPU holds the FULL-length sequence for
 *     H/d of the heads (d = the sequence's SP degree) and attends locally, with no communication.
 *   - Sec. 2.2 "Sequence Packing": a batch is a token budget of packed variable-length segments that never
 *     attend to one another.
 *   - Sec. 4.1.1 (Def. 1, SP tree) and Sec. 4.1.2 "Tree level": a GPU takes part in every node of its
 *     leaf-to-root chain, so one GPU's share mixes segments of different degrees, i.e. different head counts.
 *   - Sec. 4.1.2 "SP-backend level": the compute phase T^comp exists separately for forward and backward; this
 *     library is that phase. The paper hands it to standard softmax-attention kernels and prints no formula,
 *     so the semantics are the textbook ones:
 *         S_ij = scale * <Q[i,h], K[j,g]>  (j <= i, diagonal included; g = h / (Hq/Hkv), contiguous groups)
 *         LSE_i = ln sum_j exp(S_ij);  P_ij = exp(S_ij - LSE_i);  O[i,h] = sum_j P_ij V[j,g]
 *         dQ, dK, dV = gradients of sum(O * dO); dK/dV are summed over the Hq/Hkv query heads of a KV head.
 *
 * Packed layout ("ragged token-major"), head_dim D = 128 or 64 (one value per plan):
 *   segment s has L_s = cu_seqlens[s+1]-cu_seqlens[s] tokens, hq[s] query heads and hkv[s] KV heads.
 *   Q, O, dO, dQ : segment s is a contiguous [L_s, hq[s], D] block at element offset D * sum_{t<s} L_t*hq[t].
 *   K, V, dK, dV : segment s is a contiguous [L_s, hkv[s], D] block at element offset D * sum_{t<s} L_t*hkv[t].
 *   LSE          : fp32, segment s is [hq[s], L_s] at element offset sum_{t<s} L_t*hq[t]; natural log,
 *                  softmax scale included.
 *   A maximal range of consecutive segments with equal (hq, hkv) is a "run" (one tree node's samples);
 *   at most NSP_MAX_RUNS runs per plan.
 *
 * Pointers: metadata pointers (cu_seqlens, hq, hkv, opts, every out-parameter) are HOST pointers; tensor and
 * workspace pointers are DEVICE pointers on the current device, 16-byte aligned, owned by the caller.
 * The plan is owned by the library (nsp_plan_destroy frees it). Calls enqueue work on the given CUDA stream
 * (a cudaStream_t passed as void*; NULL = default stream) and return without synchronising unless stated.
 * Outputs are fully overwritten. A plan may be in use by one stream at a time.
 *
 * Errors: every function returns an NSP_* code; nothing throws, aborts or traps. Device-side problems (a bounded
 * wait that ran out) are recorded by the failing kernel in a per-plan status record that lives in device memory and in
 * mapped pinned host memory. Every call that takes the plan looks at the host copy first (a host load, no
 * synchronisation) and, once it is set, answers with that code and enqueues nothing: the failure surfaces at the
 * first call made after the failing kernel has written it. nsp_device_status synchronises and returns the record.
 * There is no CPU fallback: without a CUDA device the compute calls return NSP_ERR_CUDA.
 */
#ifndef NSP_H_
#define NSP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NSP_MAX_RUNS 32
#define NSP_HEAD_DIM 128

enum {
  NSP_OK = 0,
  NSP_ERR_INVALID_ARG = 1,    /* null pointer, bad metadata, misaligned tensor, bad dtype, bad scale */
  NSP_ERR_UNSUPPORTED = 2,    /* head_dim not 128 or 64, too many runs, tile sizes not built, counts out of range */
  NSP_ERR_ALLOC = 3,          /* host or device allocation failed (plan construction only) */
  NSP_ERR_CUDA = 4,           /* a CUDA runtime/driver call failed (including: no device) */
  NSP_ERR_DEVICE_TIMEOUT = 5, /* a bounded device-side wait expired (sticky, see nsp_device_status) */
  NSP_ERR_WORKSPACE = 6,      /* workspace pointer null/misaligned or ws_bytes too small */
  NSP_ERR_DEVICE_ASSERT = 7,  /* an index check inside a kernel failed (only the checked build, libnsp_checked.so,
                                 contains such checks; sticky like DEVICE_TIMEOUT) */
  NSP_ERR_INFEASIBLE = 8      /* nsp_route_sp_tree: no placement of the searched prefix fits the token budget */
};

enum { NSP_BF16 = 0, NSP_F32 = 1 }; /* output dtypes of the gradients */

typedef struct nsp_plan nsp_plan_t; /* opaque */

/* One work item of the in-GPU schedule. forward: head = q head, tile = q tile. backward: head = kv head,
 * tile = key tile. cost = number of inner-loop steps (see nsp_plan_tiles). */
typedef struct {
  int32_t seg, head, tile, cost;
} nsp_tile_t;

/* bm / bn: query / key tile rows (built: 128 / 128). order_version: 1. flags: 0, or NSP_PLAN_DETERMINISTIC_DQ:
 * the backward pass then adds the dQ tiles of a (segment, q head, q tile) in key-tile order (a turn counter per tile,
 * taken with the library's bounded wait), so that dQ, like O, LSE, dK and dV, comes out bit for bit the same in every
 * run and for every packing order; bwd_ws_bytes grows by 4 bytes per (q head, q tile). Without the flag the tiles
 * are added in arrival order with floating-point reductions: equal up to the rounding of an fp32 sum.
 * NSP_PLAN_ROUNDED_DQ reaches the same bitwise reproducibility without any waiting: every term a key tile adds to the
 * fp32 accumulator of dQ / softmax_scale is first rounded to a multiple of 2^-12; sums of such multiples are exact in
 * fp32 while they stay below 4096, so the order of the additions cannot change the result. The price is accuracy with
 * an ABSOLUTE quantum (at most 2^-13 of error per key tile and element, in units of dQ / softmax_scale): meant for
 * gradients of order one, as in training with normalised activations; should an accumulator element pass 4096 the sum
 * is merely no longer order-independent. Ignored when NSP_PLAN_DETERMINISTIC_DQ is set as well. */
#define NSP_PLAN_DETERMINISTIC_DQ 1
#define NSP_PLAN_ROUNDED_DQ 2
typedef struct {
  int32_t bm, bn, order_version, flags;
} nsp_plan_opts;

/*
 * Build the device-side work lists for one packed batch (the in-GPU counterpart of the paper's per-node
 * issue order, Sec. 4.2.1 "Inter-level Phase Streaming"; the paper balances across GPUs, this list balances the SMs of one GPU).
 *   forward  item (s, h, m), h in [0,hq[s]), m in [0, ceil(L_s/bm)):  cost = ceil(min(L_s,(m+1)*bm) / bn)
 *   backward item (s, g, n), g in [0,hkv[s]), n in [0, ceil(L_s/bn)): cost = (hq[s]/hkv[s]) * (ceil(L_s/bm) - floor(n*bn/bm))
 *   order: cost descending, then seg, tile, head ascending (a total order: the list is unique).
 * cu_seqlens [n_seg+1], hq [n_seg], hkv [n_seg]: host arrays, copied. Zero-length segments and n_seg == 0 are legal.
 * opts may be NULL (= {128,128,1,0}). The lists are built by kernels enqueued on `stream`.
 * Errors: INVALID_ARG (null, n_seg < 0, cu_seqlens[0] != 0, decreasing cu_seqlens, hq/hkv <= 0, hq % hkv != 0),
 * UNSUPPORTED (head_dim other than 128 or 64, > NSP_MAX_RUNS runs, unsupported tile sizes, >= 65536 segments, > 256 heads,
 * >= 65536 tiles in a segment), ALLOC, CUDA. On error *out_plan is NULL.
 */
int nsp_plan_tiles(const int32_t* cu_seqlens, const int32_t* hq, const int32_t* hkv, int32_t n_seg, int32_t head_dim,
                   const nsp_plan_opts* opts, void* stream, nsp_plan_t** out_plan);

/* Element counts of the packed tensors (q_elems: Q/O/dO/dQ; kv_elems: K/V/dK/dV; lse_elems: LSE) and the
 * workspace bytes nsp_attn_fwd / nsp_attn_bwd need. Any out pointer may be NULL. Host-only, no CUDA call. */
int nsp_plan_sizes(const nsp_plan_t* plan, int64_t* q_elems, int64_t* kv_elems, int64_t* lse_elems,
                   size_t* fwd_ws_bytes, size_t* bwd_ws_bytes);

/* Copy a work list to the host (pass 0 = forward, 1 = backward: the lists defined above, bit-exact; pass 2 = the
 * backward items in the order the backward kernel actually walks them, a permutation of pass 1 that is just as
 * unique: the (segment, kv head) groups by segment length descending, then segment, then kv head ascending; inside a
 * group the key tiles ascending. Group-major order keeps the dQ accumulator rows of a q tile in L2 while all key tiles
 * of the group add to them. Writes min(cap, n) items, stores n in *n_items (host_out may be NULL to query). The lists
 * were complete when nsp_plan_tiles returned; this call only copies. */
int nsp_plan_get(const nsp_plan_t* plan, int pass, nsp_tile_t* host_out, int64_t cap, int64_t* n_items);

/*
 * Forward (paper Sec. 4.1.2, T^comp,fwd of every node on this GPU's chain, in one launch).
 * q [q_elems] bf16, k/v [kv_elems] bf16 (device, read-only); o [q_elems] bf16 and lse [lse_elems] fp32 (device,
 * written). softmax_scale: finite, > 0. ws / ws_bytes: device workspace of at least fwd_ws_bytes (may be NULL
 * when that is 0). Errors: INVALID_ARG, WORKSPACE, CUDA, DEVICE_TIMEOUT (sticky status from an earlier call).
 */
int nsp_attn_fwd(const nsp_plan_t* plan, const void* q, const void* k, const void* v, void* o, float* lse,
                 float softmax_scale, void* ws, size_t ws_bytes, void* stream);

/*
 * Backward (paper Sec. 4.1.2, T^comp,bwd). Inputs: q, k, v, o, d_o (bf16) and lse (fp32) as produced by
 * nsp_attn_fwd. Outputs: dq [q_elems], dk/dv [kv_elems] in dq_dtype / dkv_dtype (NSP_BF16 or NSP_F32);
 * dk/dv hold the sum over the hq/hkv query heads that share a KV head on THIS GPU (with a replicated KV head
 * at high degree the cross-GPU sum belongs to the epilogue collective, outside this library).
 * ws: at least bwd_ws_bytes, 256-byte aligned; contents undefined afterwards.
 * Errors: as nsp_attn_fwd.
 */
int nsp_attn_bwd(const nsp_plan_t* plan, const void* q, const void* k, const void* v, const void* o, const void* d_o,
                 const float* lse, void* dq, void* dk, void* dv, int dq_dtype, int dkv_dtype, float softmax_scale,
                 void* ws, size_t ws_bytes, void* stream);

/*
 * (No counterpart in the paper: an addition for callers that are not allowed to allocate.)
 * nsp_attn_bwd without a caller-provided workspace. Some callers cannot supply one: an executor that handed all
 * device memory to its own planner or caching pool at start-up has no way to obtain a transient q-sized fp32
 * buffer mid-iteration, because cudaMalloc would synchronise the device, may fail once the pool owns the memory,
 * and is banned inside some schedulers. For them the scratch (fp32 dQ accumulator + delta) is a fixed array of
 * NSP_STATIC_WS_BYTES inside the library image. The driver reserves that memory on a GPU when it loads the module that
 * holds the array: with the default lazy module loading that is the FIRST call of this function on the device (which
 * looks up the array's device address with cudaGetSymbolAddress, that device being current), with eager loading
 * (CUDA_MODULE_LOADING=EAGER) it is library load; the GPU then holds it until the process exits. So make that first
 * call (any small batch will do) at start-up, before the caller's pool takes the remaining memory and before any
 * stream capture begins: made later it may fail with NSP_ERR_CUDA for lack of memory, and it may synchronise.
 * From the second call on a device, the call makes no cudaMalloc / cudaFree, calls no allocating routine and changes
 * nothing about the device's free memory.
 * Arguments, outputs and results are those of nsp_attn_bwd (same kernels); inputs and outputs are still the caller's.
 * Limit: plans whose bwd_ws_bytes (see nsp_plan_sizes; roughly 4 * q_elems + 4 * lse_elems bytes) exceed
 * NSP_STATIC_WS_BYTES are rejected with NSP_ERR_WORKSPACE and nothing is enqueued.
 * The array is shared by all calls and keeps the previous call's contents: the accumulator part is cleared on
 * `stream` at the start of each call, and two calls whose device work overlaps (other streams or host threads) race
 * on it -- serialise them.
 * Errors: INVALID_ARG, WORKSPACE (batch too large), CUDA, DEVICE_TIMEOUT, as nsp_attn_bwd.
 */
#define NSP_STATIC_WS_BYTES (32u * 1024u * 1024u)
int nsp_attn_bwd_static(const nsp_plan_t* plan, const void* q, const void* k, const void* v, const void* o,
                        const void* d_o, const float* lse, void* dq, void* dk, void* dv, int dq_dtype, int dkv_dtype,
                        float softmax_scale, void* stream);

/*
 * One forward + backward pass with HOST buffers (paper Sec. 4.1.2: T^comp,fwd + T^comp,bwd of this GPU's chain, as a
 * caller sees it whose tensors live in host memory): nsp_attn_fwd followed by nsp_attn_bwd on device copies that this
 * call makes and reads back.
 * h_q, h_do [q_elems] bf16, h_k, h_v [kv_elems] bf16: host, read. h_o [q_elems] bf16, h_lse [lse_elems] fp32, h_dq
 * [q_elems] in dq_dtype, h_dk / h_dv [kv_elems] in dkv_dtype: host, written. Pinned (page-locked) host memory lets
 * the copies run asynchronously; with pageable memory they still work but the call blocks while they are staged.
 * dev_ws: device memory of at least nsp_plan_step_host_ws_bytes(plan, dq_dtype, dkv_dtype) bytes, 256-byte aligned,
 * owned by the caller: it holds the nine device tensors and the backward workspace; contents undefined afterwards.
 * The copies run on a second stream owned by the plan (created, with six events, at the first call on the plan: make
 * that call outside any stream capture), ordered with events against `stream`: dO travels to the device while the
 * forward pass runs, O and LSE travel back while the backward pass runs; exposed are the copies of Q, K, V before the
 * forward pass and of dQ, dK, dV after the backward pass. The call returns without waiting; the host outputs are
 * complete once `stream` has passed everything this call enqueued on it (synchronise `stream`), and the host inputs
 * must stay unchanged until then. Two calls on the same plan must not overlap from different host threads.
 * Errors: INVALID_ARG (null pointer, dtype), WORKSPACE (dev_ws missing, misaligned or too small), CUDA,
 * DEVICE_TIMEOUT (sticky status), and whatever nsp_attn_fwd / nsp_attn_bwd return.
 */
int nsp_plan_step_host_ws_bytes(const nsp_plan_t* plan, int dq_dtype, int dkv_dtype, size_t* bytes);
int nsp_attn_step_host(nsp_plan_t* plan, const void* h_q, const void* h_k, const void* h_v, const void* h_do, void* h_o,
                       float* h_lse, void* h_dq, void* h_dk, void* h_dv, int dq_dtype, int dkv_dtype,
                       float softmax_scale, void* dev_ws, size_t dev_ws_bytes, void* stream);

/*
 * Tree-level recomputation (paper Sec. 4.2.2 "Tree-Level Recomputation"): the backward pass of a shard in which the
 * attention output of some segments was not kept after the forward pass.
 *
 * nsp_recompute_mark derives the save / recompute marking of this GPU's segments from an activation budget, the way
 * the paper's executor walks its tree: segments (cu_seqlens [n_seg + 1], hq [n_seg], as for nsp_plan_tiles; all
 * host) are visited from the upper levels down (level[s], host, larger =
 * closer to the root, e.g. the SP degree of the segment's node; inside a level the segment that is more expensive to
 * recompute first, cost = hq * L(L+1)/2), the bytes a saved segment keeps alive (its O slice in bf16 and its LSE in
 * fp32: L * hq * (2 * head_dim + 4)) are accumulated, and from the first segment that no longer fits under
 * budget_bytes on, everything is marked for recomputation. recompute (host, [n_seg], written): 0 = save,
 * 1 = recompute. saved_bytes (may be NULL): bytes of the saved segments. Host-only, no CUDA call.
 * Errors: INVALID_ARG (null pointer, negative size or budget, decreasing cu_seqlens, hq <= 0).
 *
 * nsp_attn_bwd_recompute is nsp_attn_bwd with such a marking (recompute: host, [n_seg]; if it is pinned memory it
 * must stay unchanged until the stream has passed the call). For a marked segment the contents of o and lse are
 * never read: a forward launch restricted to the marked segments recomputes their LSE and forms
 * delta = rowsum(dO o O) from the accumulator in the same kernel, so the recomputed O never travels to memory; for
 * the other segments o and lse are used as in nsp_attn_bwd. Outputs as nsp_attn_bwd. ws: at least
 * nsp_plan_recompute_ws_bytes (the backward workspace plus an LSE copy and the flags), 256-byte aligned.
 * Errors: as nsp_attn_bwd.
 */
int nsp_recompute_mark(const int32_t* cu_seqlens, const int32_t* hq, const int32_t* level, int32_t n_seg,
                       int32_t head_dim, int64_t budget_bytes, uint8_t* recompute, int64_t* saved_bytes);
int nsp_plan_recompute_ws_bytes(const nsp_plan_t* plan, size_t* bytes);
int nsp_attn_bwd_recompute(const nsp_plan_t* plan, const uint8_t* recompute, const void* q, const void* k,
                           const void* v, const void* o, const void* d_o, const float* lse, void* dq, void* dk,
                           void* dv, int dq_dtype, int dkv_dtype, float softmax_scale, void* ws, size_t ws_bytes,
                           void* stream);

/*
 * Planner (paper Sec. 4.1.2 "Routing Objective and Cost Model" and Sec. 4.1.3, Algorithm 1 "Prefix-Completion SP-Tree
 * Routing").
 * Host only, no CUDA call.
 *
 * The SP tree is the full binary tree over P = 2^(n_levels-1) GPUs: node (l, i) covers GPUs [i*2^l, (i+1)*2^l) and
 * runs its samples at SP degree 2^l.
 *
 * nsp_cost_table fills cost_out [n_samples * n_levels] (row j, column l: the load, in nanoseconds, that sample j
 * puts on EVERY GPU of a level-l node, forward + backward) from profiled coefficients, level by level as the paper's
 * cost model: compute = L(L+1)/2 causal pairs x hq/2^l local q heads x tcomp_ns[l * NSP_COST_BUCKETS + b] (profiled
 * nanoseconds per pair and head at level l for the length class b = clip(floor(log2 L), 5, 20) - 5); prologue +
 * epilogue = (L/d)(d-1)/d tokens x 4 * head_dim * (2 hq + 2 hkv) bytes (Q, K, V in and O out, forward and backward,
 * bf16) / link_gbs[l] (GB/s of the fabric a level-l group communicates over; unused for l = 0); non-attention
 * work = L/d tokens x other_ns_per_token. The sum is rounded to the nearest integer. hq, hkv: heads of the whole
 * model. Errors: INVALID_ARG.
 *
 * nsp_route_sp_tree routes a batch: samples are visited by nonincreasing length (equal lengths keep their order);
 * the first prefix_k are placed by a beam search over all tree nodes (root first, left to right; with monotone != 0
 * a sample may not sit above the level of the previous, longer one), dropping states in which a GPU's token load
 * Tok_p = sum of L/d exceeds b_tok and keeping the beam_w states with the smallest critical load max_p C_p (ties:
 * order of generation); every surviving state is then completed greedily, each remaining sample going to the
 * least-loaded single-GPU leaf that stays within b_tok, or to the leaf with the smallest token load when none
 * does; the completed state with the smallest critical load is returned, states within the budget first.
 * Outputs (host): level_out / index_out [n_samples] = the node of every sample; load_out [P] = C_p; tok_out [P] =
 * Tok_p in units of 1/P token; feasible_out = 1 if every GPU is within b_tok (the last three may be NULL).
 * Cost is O(prefix_k * beam_w * (2P-1) * P). Errors: INVALID_ARG (negative sizes, lengths or costs, n_levels not
 * in 1..11, beam_w < 1), INFEASIBLE (no token-feasible placement of the prefix; nothing is written).
 */
#define NSP_COST_BUCKETS 16
int nsp_cost_table(const int32_t* lengths, int32_t n_samples, int32_t n_levels, int32_t hq, int32_t hkv,
                   int32_t head_dim, const double* tcomp_ns, const double* link_gbs, double other_ns_per_token,
                   int64_t* cost_out);
int nsp_route_sp_tree(const int32_t* lengths, const int64_t* cost, int32_t n_samples, int32_t n_levels,
                      int32_t prefix_k, int32_t beam_w, int64_t b_tok, int32_t monotone, int32_t* level_out,
                      int32_t* index_out, int64_t* load_out, int64_t* tok_out, int32_t* feasible_out);

/*
 * Layout steps of the Ulysses all-to-all around the attention compute (paper Sec. 2.1; the prologue and epilogue
 * phases of a tree node, Sec. 4.1.2). The exchange itself (NCCL send / receive between the GPUs of the node) is issued
 * by the caller; see ulysses.py for the schedule. Tensors are device pointers, rows of head_dim elements of dtype
 * NSP_BF16 or NSP_F32, head_dim * element size a multiple of 16 bytes, pointers 16-byte aligned; first_head is a
 * host array [n_blocks], n_blocks <= NSP_A2A_MAX_PEERS.
 *
 * nsp_a2a_gather_heads: src [tokens, heads, head_dim] (this GPU's token slice, all heads) -> dst [n_blocks][tokens,
 * heads_per_block, head_dim], block p = heads [first_head[p], first_head[p] + heads_per_block): the contiguous block
 * peer p receives. Blocks may overlap (a KV head replicated over several peers).
 * nsp_a2a_scatter_heads: the inverse, src [n_blocks][tokens, heads_per_block, head_dim] -> dst [tokens, heads,
 * head_dim]; where several blocks carry the same head (partial dK / dV of a replicated KV head) they are added in
 * block order in fp32; heads no block carries are left untouched.
 * Errors: INVALID_ARG, UNSUPPORTED (row size not a multiple of 16 bytes), CUDA.
 */
#define NSP_A2A_MAX_PEERS 64
/*
 * nsp_a2a_gather_heads_to: the send side of the prologue fused with the exchange. The same head gather as
 * nsp_a2a_gather_heads, but block p is not staged: its rows are stored straight into dst_base[p], the packed
 * attention buffer [t_full, heads_per_block, head_dim] the receiving GPU's nsp_attn_fwd reads (a peer's memory mapped
 * into this process, or a local buffer). src holds the token slices of n_samples samples one after the other;
 * sample_off (DEVICE, int64 [n_samples + 1], sample_off[0] = 0, last = tokens) gives their rows in src, and
 * dst_row (DEVICE, int64 [n_blocks * n_samples]) the row in dst_base[p] where this GPU's slice of sample j starts
 * (entry p * n_samples + j). dst_base and first_head are host arrays [n_blocks]. The stores are plain 16-byte stores
 * issued by the library's own kernel; the receiver may read its buffer once it has synchronised with this stream
 * (an event or a barrier between the GPUs is the caller's). Errors as nsp_a2a_gather_heads.
 */
int nsp_a2a_gather_heads_to(const void* src, void* const* dst_base, const int64_t* dst_row, const int64_t* sample_off,
                            int32_t n_samples, int64_t tokens, int32_t heads, int32_t heads_per_block, int32_t n_blocks,
                            int32_t head_dim, int32_t dtype, const int32_t* first_head, void* stream);
int nsp_a2a_gather_heads(const void* src, void* dst, int64_t tokens, int32_t heads, int32_t heads_per_block,
                         int32_t n_blocks, int32_t head_dim, int32_t dtype, const int32_t* first_head, void* stream);
int nsp_a2a_scatter_heads(const void* src, void* dst, int64_t tokens, int32_t heads, int32_t heads_per_block,
                          int32_t n_blocks, int32_t head_dim, int32_t dtype, const int32_t* first_head, void* stream);

/* Read the device status record {code, item, where, aux}; code 0 = healthy. Synchronises the device. */
int nsp_device_status(const nsp_plan_t* plan, int32_t out[4]);

/* Failure-detection self test: enqueues a one-warp kernel that waits, with the library's bounded wait, on a barrier
 * nothing arrives at. After limit_clk SM cycles (1 .. 2^31; a million is well under a millisecond) the wait gives
 * up and the kernel records NSP_ERR_DEVICE_TIMEOUT in the plan's status word, the way a stalled attention kernel
 * would; nothing traps, the context stays usable, other plans are unaffected. nsp_device_status then reads
 * {NSP_ERR_DEVICE_TIMEOUT, -1, 90, limit_clk / 1024} and the plan answers every later call with that code.
 * Errors: INVALID_ARG, CUDA, or the plan's sticky status. */
int nsp_selftest_wait_timeout(const nsp_plan_t* plan, int64_t limit_clk, void* stream);

/* How long a device-side wait of this plan's kernels may take before it gives up, in SM clocks (default 4e9, about
 * two seconds; at least 1000). Every wait on a barrier inside the kernels is bounded by it; when one runs out the kernel
 * records NSP_ERR_DEVICE_TIMEOUT with the work item and the place, all its roles unwind and the launch ends. Errors:
 * INVALID_ARG. */
int nsp_plan_set_wait_limit(nsp_plan_t* plan, int64_t sm_clocks);

#ifdef NSP_CHECKED
/* Checked build only (libnsp_checked.so, compiled with -DNSP_CHECKED: every index a kernel computes for a global
 * access is verified first, a failing one is recorded as NSP_ERR_DEVICE_ASSERT and the access skipped). Test switch for
 * the failure path: with enable != 0 the next forward launch leaves out one V tile load, so that the waits behind it
 * run out (use a small nsp_plan_set_wait_limit); nothing faults, the launch ends with NSP_ERR_DEVICE_TIMEOUT. */
int nsp_checked_withhold_load(nsp_plan_t* plan, int enable);
#endif

/* Kernels of the path, for nsp_plan_kernel_ms. */
enum {
  NSP_KERNEL_FWD = 0,
  NSP_KERNEL_BWD_PRE = 1,
  NSP_KERNEL_BWD_MAIN = 2,
  NSP_KERNEL_BWD_POST = 3,
  NSP_KERNEL_BWD_FIRST = 4, /* the backward kernel for the first 128 tokens of every segment */
  NSP_KERNEL_FWD_FIRST = 5, /* the forward kernel for the first 128 tokens of every segment */
  NSP_KERNEL_COUNT = 6
};

/* Measurement aid (the paper's cost model is fed by offline profiles of the compute phase, Sec. 4.1.2): when
 * enabled, every later nsp_attn_fwd / nsp_attn_bwd on this plan brackets each of its kernels with a pair of CUDA
 * events recorded on the launching stream. Errors: INVALID_ARG (null plan), CUDA. */
int nsp_plan_set_profiling(nsp_plan_t* plan, int enable);

/* Device time in milliseconds of the most recent launch of kernel `kernel_id` (NSP_KERNEL_*) on this plan.
 * Waits for that launch to finish. Errors: INVALID_ARG (profiling off, kernel not launched yet, bad id), CUDA. */
int nsp_plan_kernel_ms(const nsp_plan_t* plan, int kernel_id, float* ms);

/* Number of kernel launches the library has enqueued so far in this process (all plans). */
int64_t nsp_launch_count(void);

/* Free the plan (device lists, tables, status word). NULL is a no-op. */
int nsp_plan_destroy(nsp_plan_t* plan);

const char* nsp_status_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* NSP_H_ */
