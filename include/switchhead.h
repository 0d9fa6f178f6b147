/*
 * switchhead.h - C ABI of the B200 (sm_100a) forward pass of one SwitchHead attention layer.
 *
 * The layer (paper Sec. 2.2): for an input x [B, T, d_model] and each of n_heads heads h,
 *   source gate       s_S^h = sigmoid(x W_S^h),  destination gate  s_D^h = sigmoid(x W_D^h)
 *   selections        E_S^h(t), E_D^h(t) = arg top-k over the E experts, per token
 *   values            V^h[t] = sum_{e in E_S^h(t)} s_S^h[t,e] * x[t] W_V^{h,e}
 *   queries / keys    Q^h = x W_Q^h,  K^h = x W_K^h           (one dense pair per head)
 *   attention         A^h = softmax(Q^h K^h^T / sqrt(d_head)) (Eq. 1), causal: key s <= query t
 *   output            y[t] = sum_h sum_{e in E_D^h(t)} s_D^h[t,e] * (A^h V^h)[t] W_O^{h,e}
 * Top-k is taken on the pre-sigmoid logits; equal logits go to the lower expert index.
 * Selected gates are not renormalised.  Batch elements are independent sequences.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless the comment says "host".
 *   - Arrays are dense, row-major, in the layouts stated per argument.
 *   - `stream` is a cudaStream_t passed as void*; NULL is the default stream.  The device work
 *     of a call is ordered on that stream: it starts after everything enqueued there before
 *     the call and is complete before anything enqueued there after it.  The bf16 forward pass
 *     also uses two non-blocking streams the layer owns (the dense Q/K projection runs on them
 *     beside the gate and sort kernels, forked from and joined back into `stream` with
 *     events), which matters to a caller that captures `stream` into a graph or gives it a
 *     priority.  No call synchronises the device unless its comment says so.
 *   - The release library reads nothing from the environment.
 *   - Functions returning int give SH_OK (0) or a negative SH_ERR_* code; sh_last_error()
 *     then holds a readable reason (thread-local, host string owned by the library).
 *   - The library owns only the handle.  x, out, the source weights and the workspace
 *     belong to the caller.  sh_forward / sh_gate_topk allocate nothing.
 *   - Inputs must be finite.  There is no CPU fallback: without a CUDA device every
 *     launching call fails with SH_ERR_CUDA.
 */
#ifndef SWITCHHEAD_H_
#define SWITCHHEAD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sh_layer sh_layer;

enum { SH_F32 = 0, SH_BF16 = 1 };

enum {
  SH_OK = 0,
  SH_ERR_INVALID_ARG = -1,
  SH_ERR_UNSUPPORTED = -2,
  SH_ERR_NOT_CONFIGURED = -3,
  SH_ERR_WORKSPACE = -4,
  SH_ERR_CUDA = -5,
  SH_ERR_TIMEOUT = -6, /* a bounded device-side wait ran out (reported by sh_last_status) */
  SH_ERR_BOUNDS = -7   /* an index check of the debug library failed (sh_last_status), or
                          sh_check_guards found a guard behind a workspace buffer overwritten */
};

/* Identifiers for sh_debug_buffer. */
enum {
  SH_BUF_Q = 0,      /* [B, H, T, D]  queries, pre-multiplied by log2(e)/sqrt(D)            */
  SH_BUF_K = 1,      /* [B, H, T, D]                                                        */
  SH_BUF_V = 2,      /* [B, H, T, D]  gate-weighted sum of the selected value experts       */
  SH_BUF_AHAT = 3,   /* [B*T, H, D]   attention read-out (A^h V^h)[t]                        */
  SH_BUF_IDX = 4,    /* [2, N, H, k]  int32                                                 */
  SH_BUF_GATE = 5,   /* [2, N, H, k]  fp32                                                  */
  SH_BUF_OFFSETS = 6,/* [2, H, E+1]   int32                                                 */
  SH_BUF_LISTS = 7   /* [2, H, N*k]   int32                                                 */
};

/* Create a layer description.  Host-only, no CUDA call.
 * Requires 1 <= k <= n_experts <= 32, n_heads >= 1, 1 <= d_head <= 256, d_model a positive multiple of 64.
 * (bf16 storage with d_head above 128 - the paper's 132 and 168 - runs every stage on the CUDA-core
 * kernels: correct and slow, the plain layer only; the tensor-core kernels serve d_head <= 128.)
 * d_head is stored padded with zero columns to 64, 128 or 256 (bf16 storage) or to 32, 64, 128 or 256 (fp32): the padding changes no result (the scale stays 1/sqrt(d_head)),
 * it costs the time of the padded size, and the Q, K, V, Ahat debug buffers have the padded
 * width.  Returns NULL on error (see sh_last_error). */
sh_layer* sh_create(int d_model, int n_heads, int d_head, int n_experts, int k);

/* The "Shared Selection" variant of the paper's appendix: one gate serves the source and the
 * destination side, so the output experts of a token are the ones its value projection
 * selected, with the same scores; one top-k and one bucket sort per head instead of two.
 * Same arguments and limits as sh_create.  sh_set_weights takes the gate as Ws / bias_s and
 * wants NULL for Wd and bias_d; the two sides of sh_gate_topk's outputs (and of the
 * idx / gate / offsets / lists debug buffers' first half) are then equal. */
sh_layer* sh_create_shared(int d_model, int n_heads, int d_head, int n_experts, int k);

/* SwitchHead layer whose query and / or key projections are experts too (Sec. 2.2 writes K^h and
 * Q^h as expert sums like V^h; the paper's ablation over which projections are experts keeps them
 * dense in the final model, which is what sh_create builds).  moe_k != 0: K^h[t] = sum over the
 * experts the SOURCE side of token t selected, weighted by its scores, of x[t] W_K^{h,e} (the
 * selection the value projection uses); moe_q != 0: Q^h[t] likewise with the DESTINATION side's
 * selection (the one the output projection uses).  sh_set_weights then takes Wq as [H, E, d_model,
 * d_head] (moe_q) and Wk as [H, E, d_model, d_head] (moe_k) instead of [H, d_model, d_head].
 * shared_selection != 0: one gate for both sides, as sh_create_shared (keys and queries then use the
 * same selection).  SH_F32 takes every shape.  SH_BF16 (tensor-core path): an expert projection of
 * keys / queries runs on the pair-tiled value-expert kernel, so sh_configure wants k = 2, 2..8
 * experts, d_head in 65..128 and, when only one of the two is an expert projection, an even number
 * of heads; it refuses other shapes.  sh_set_rope refuses such a layer.  Other arguments and limits
 * as sh_create. */
sh_layer* sh_create_moe_qk(int d_model, int n_heads, int d_head, int n_experts, int k, int moe_q, int moe_k,
                           int shared_selection);

/* Dense multi-head attention comparator (Eq. 1-2) built from the same kernels: every head
 * has one dense W_V and W_O and there are no gates.  Used only to time a parameter-matched
 * dense layer beside SwitchHead.  Weights are passed to sh_set_weights with n_experts = 1
 * and Ws = Wd = NULL.  Returns NULL on error. */
sh_layer* sh_create_dense(int d_model, int n_heads, int d_head);

/* Fix the storage type and the problem size.  dtype SH_F32: x and weights fp32, all
 * arithmetic fp32 on CUDA cores.  dtype SH_BF16: x and weights bf16, tensor-core products
 * with fp32 accumulation, fp16 intermediates (Q, K, V, P, A^h V^h); requires d_model a
 * multiple of 128.  `out` is fp32 in both cases.
 * batch*seq*n_heads*k must be below 2^31.  Invalidates workspace and weights. */
int sh_configure(sh_layer* layer, int dtype, int batch, int seq);

/* The same with a Transformer-XL context (the paper's main models, Sec. 3 "Experiments" and the
 * appendix on resource usage: the attention of a chunk of T tokens spans C*T keys, the extra
 * (C-1)*T being a cache of the previous chunk(s); the paper uses C = 2).  x passed to sh_forward is
 * then [B, cache_len + seq, d_model]: for every sequence the cached tokens - the INPUT this layer
 * received for the previous chunk, which the caller keeps - followed by the current chunk.  Keys,
 * values and the source-side gate with its expert selection are computed for all cache_len + seq
 * tokens; queries, the destination-side gate and the output for the chunk's tokens only, each of
 * which sees the whole cache and the chunk up to itself.  out is [B, seq, d_model].
 * bf16 storage: cache_len and seq must be multiples of 128 (else SH_ERR_UNSUPPORTED).
 * Scores are q.k / sqrt(d_head) unless sh_set_xl_positions adds Transformer-XL's relative-position
 * term.  sh_set_rope is refused for a layer with a cache; sh_gate_topk and the debug
 * buffers cover all cache_len + seq tokens.  cache_len = 0 is sh_configure. */
int sh_configure_xl(sh_layer* layer, int dtype, int batch, int seq, int cache_len);

/* The relative-position term of Transformer-XL (the positional encoding of the paper's main models;
 * the paper cites it and does not restate it) for the fp32 configuration:
 *   score[t, s] = ( (q_t + u^h) . k_s  +  (q_t + v^h) . r^h_{t-s} ) / sqrt(d_head),
 *   r^h_dist = emb(dist) Wr^h,   emb(dist) = [sin(dist w_0..), cos(dist w_0..)], w_i = 10000^(-2i/d_model)
 * where t and s are positions in [cache; chunk] and only keys s <= t are visible.
 *   Wr [H, d_model, d_head] fp32, u, v [H, d_head] fp32 (NULL: zero).  Wr = NULL switches the term off.
 * Builds the distance tables for the configured sequence length in the workspace (asynchronously
 * on `stream`); valid until the next sh_configure / sh_set_workspace.  Wr, u, v are fp32 for both
 * storage types.  fp32 configuration: with and without a cache; the CUDA-core attention kernel
 * evaluates both terms.  bf16 storage: for a layer with a cache (sh_configure_xl, the setting of the
 * paper's XL models; else SH_ERR_UNSUPPORTED): every pass computes u.k per key and a score bias
 * [B, H, seq, cache_len + seq] fp16 = Q R^T (shifted from distance order to key order) + v.r + u.k
 * with a tensor-core GEMM, and the attention kernel adds it to its score tiles.
 * SH_ERR_UNSUPPORTED while rotary embeddings are on. */
int sh_set_xl_positions(sh_layer* layer, const float* Wr, const float* u, const float* v, void* stream);

/* Bytes of workspace sh_set_workspace needs for the current configuration (0 if not
 * configured). */
size_t sh_workspace_bytes(const sh_layer* layer);

/* Hand the layer a caller-owned device buffer of at least sh_workspace_bytes() bytes,
 * aligned to 256 bytes.  It must stay valid until sh_destroy or the next sh_configure.
 * Holds repacked weights, intermediates, token lists and the device status word. */
int sh_set_workspace(sh_layer* layer, void* workspace, size_t bytes);

/* Repack the weights into the workspace (asynchronously on `stream`); the caller may free
 * or overwrite its copies once the stream has passed this point.  Element type = dtype of
 * sh_configure.
 *   Wq, Wk  [H, d_model, d_head]
 *   Wv      [H, E, d_model, d_head]
 *   Wo      [H, E, d_head, d_model]
 *   Ws, Wd  [H, d_model, E]      source-side / destination-side gate weights
 *   bias_s, bias_d  [H, E] fp32 or NULL: optional additive gate-logit bias, z = x W + b.
 *                   The paper has no bias (NULL); it exists for skew-routed test workloads. */
int sh_set_weights(sh_layer* layer, const void* Wq, const void* Wk, const void* Wv,
                   const void* Wo, const void* Ws, const void* Wd, const float* bias_s,
                   const float* bias_d, void* stream);

/* Attention mask.  causal != 0 (the default): the language-model setting, key s is visible to
 * query t iff s <= t.  causal == 0: every key of the sequence is visible (the paper's ListOps
 * classifier uses SwitchHead without autoregressive masking).  Host-only; takes effect with
 * the next sh_forward. */
int sh_set_causal(sh_layer* layer, int causal);

/* Rotary position embeddings on the queries and keys (the paper's appendix "RoPE Positional
 * Encodings": square causal attention without a cache, RoPE as in RoFormer).  Token t of a
 * sequence sits at position t; the feature pair (2i, 2i+1) of its query and key vectors of
 * every head is rotated by the angle t * base^(-2i/d_head) before the attention scores are
 * taken; values are not rotated.  base > 0 switches it on (10000 is RoFormer's value) and
 * writes the (cos, sin) table for the configured sequence length into the workspace,
 * asynchronously on `stream`; base == 0 switches it off (the default, and the state after
 * every sh_configure and sh_set_workspace).  Needs a configured layer with its workspace (else
 * SH_ERR_NOT_CONFIGURED) and an even d_head. */
int sh_set_rope(sh_layer* layer, double base, void* stream);

/* The whole forward pass (gates + top-k + bucket sort, Q/K projections, value experts,
 * causal attention, output experts with the gate-weighted sum) of x [B, T, d_model] into
 * out [B, T, d_model] fp32 (with a cache, sh_configure_xl: x [B, cache_len + T, d_model]).  Both are device pointers aligned to 16 bytes (else
 * SH_ERR_INVALID_ARG).  out is fully overwritten.  Enqueues kernels only. */
int sh_forward(sh_layer* layer, const void* x, void* out, void* stream);

/* Kernel slots of sh_forward_stamped. */
enum {
  SH_STAMP_GATE = 0,   /* gate logits + top-k (+ the bucket sort when it is fused into this kernel) */
  SH_STAMP_SORT = 1,   /* bucket sort as a kernel of its own                                        */
  SH_STAMP_QK_A = 2,   /* dense Q/K projection: the grid launched ahead of the gate kernel (or the only grid) */
  SH_STAMP_QK_B = 3,   /* ... the grid launched behind the sort, when the projection is split        */
  SH_STAMP_V = 4,      /* value experts                                                              */
  SH_STAMP_ATTN = 5,   /* attention                                                                  */
  SH_STAMP_O = 6,      /* output experts + gate-weighted sum                                         */
  SH_STAMP_COUNT = 7
};

/* Measurement aid: sh_forward, launched exactly as sh_forward launches it (same kernels, streams
 * and launch attributes), with every kernel of the bf16 path writing three device-clock stamps
 * (%globaltimer, nanoseconds): `resident` = its first CTA running, `start` = its first CTA past
 * the wait for the kernel it depends on, `end` = its last CTA done.  Waits for `stream`, then
 * fills the HOST array stamps[3][SH_STAMP_COUNT] = {resident[], start[], end[]}.  A kernel that
 * did not run in this pass (and every kernel of the fp32 configuration, whose CUDA-core kernels
 * carry no stamps) leaves resident = start = UINT64_MAX and end = 0.  The spans of kernels that
 * overlap in time may be subtracted from one another: they share one clock. */
int sh_forward_stamped(sh_layer* layer, const void* x, void* out, void* stream, uint64_t* stamps);

/* Measurement aid: sh_forward with CUDA events recorded on `stream` at the stage boundaries;
 * waits for the stream, then writes to the HOST array stage_ms[6] the milliseconds of
 * {gate + top-k + sort, Q/K projection, value experts, attention, output experts, whole
 * pass}.  To give the boundaries a meaning this call serialises the pass: ordinary launches on
 * one stream, no kernel overlapping the next, so the stage times add up to MORE than a
 * sh_forward takes; sh_forward_stamped shows what each kernel costs inside the real pass.
 * Creates and destroys its events, so unlike sh_forward it must not be stream-captured. */
int sh_forward_timed(sh_layer* layer, const void* x, void* out, void* stream, float* stage_ms);

/* Gate stage alone, with its results exposed (any output pointer may be NULL):
 *   idx     [2, N, H, k] int32  selected experts; side 0 = source, 1 = destination;
 *                               in rank order (largest logit first, ties lower index first)
 *   gate    [2, N, H, k] fp32   sigmoid of the selected logits, same order
 *   offsets [2, H, E+1]  int32  exclusive scan of the per-expert token counts
 *   lists   [2, H, N*k]  int32  token ids grouped by expert, ascending within a group:
 *                               group e of (side, h) is lists[side,h,offsets[e]:offsets[e+1]]
 * N = batch*seq. */
int sh_gate_topk(sh_layer* layer, const void* x, int32_t* idx, float* gate, int32_t* offsets,
                 int32_t* lists, void* stream);

/* (No counterpart in the paper: an addition for callers that cannot allocate device memory.)
 * Some callers run where cudaMalloc is not an option - inside a memory pool they do not own,
 * in a process whose allocations are fixed at start-up, or simply without a workspace to
 * hand over.  This entry point runs the gate + top-k + bucket-sort stage (the same kernels
 * as sh_gate_topk on the CUDA cores) without a layer handle and without any allocation:
 * its scratch memory - the per-block selection histograms, the gate values in list order
 * and the row-tile table the sort kernel emits - lives in fixed arrays inside the library
 * (about 2.3 MB on every GPU that loads it, held until the process exits).  It calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *   dtype    SH_F32 or SH_BF16: element type of x and w_gate
 *   x        [n_tokens, d_model]
 *   w_gate   [2*n_heads*n_experts, d_model]: one ROW per gate column, row (side*H + h)*E + e
 *            (side 0 = source); i.e. W_S^h and W_D^h transposed and stacked
 *   bias     [2*n_heads*n_experts] fp32 added to the logits, or NULL
 *   idx, gate, offsets, lists: as for sh_gate_topk (all required here)
 * Limits: n_tokens <= 16384, 2*n_heads*n_experts <= 256, n_tokens*n_heads*k <= 262144,
 * n_experts <= 32, and n_heads*k small enough for the sort kernel's 48 KB of shared memory;
 * anything larger is refused with SH_ERR_UNSUPPORTED and a message naming the limit.
 * The first call on a device looks up the arrays' device addresses (a host-side set-up
 * step), so make that first call outside any stream capture.  All calls on a device share
 * the arrays, which keep the previous call's contents: nothing in them needs clearing
 * between calls (each call overwrites what it reads), but two calls whose kernels overlap
 * on the GPU - different streams, or different host threads - race on them; serialise them. */
int sh_noalloc_gate_topk(int dtype, int n_tokens, int d_model, int n_heads, int n_experts, int k,
                         const void* x, const void* w_gate, const float* bias, int32_t* idx,
                         float* gate, int32_t* offsets, int32_t* lists, void* stream);

/* Backward pass, fp32 configuration of the plain layer (sh_create + sh_configure(SH_F32): two gates,
 * dense Q/K, no cache, no positional term; anything else: SH_ERR_UNSUPPORTED).  The paper gives no
 * backward formulas - its training differentiates the forward equations of Sec. 2.2 automatically -
 * so this is the chain rule for those equations with the expert selection held fixed.  Call it after
 * sh_forward(layer, x, ...) on the SAME x (it reads the Q, K, V, Ahat, selections and gates that pass
 * left in the workspace; otherwise SH_ERR_NOT_CONFIGURED).  dout [batch, seq, d_model] fp32 = dL/dout.
 * Every result is a device buffer of the caller, fp32, OVERWRITTEN: dx [batch, seq, d_model]; dWq, dWk
 * [H, d_model, d_head]; dWv [H, E, d_model, d_head]; dWo [H, E, d_head, d_model]; dWs, dWd [H, d_model, E]
 * (the layouts sh_set_weights takes).  CUDA-core kernels with fp32 atomics: sums over tokens arrive in
 * any order, so two calls agree to rounding, not bit for bit.  Work enqueued on `stream`. */
int sh_backward(sh_layer* layer, const void* x, const float* dout, float* dx, float* dWq, float* dWk,
                float* dWv, float* dWo, float* dWs, float* dWd, void* stream);

/* Device pointer and size of an intermediate buffer inside the workspace (contents are
 * those of the last sh_forward / sh_gate_topk once the stream has drained).  Element type:
 * fp32 for SH_F32, fp16 for SH_BF16 (Q, K, V, AHAT); int32 / fp32 for the gate buffers.
 * The offsets and lists buffers hold what the last call left there: after sh_gate_topk the
 * per-(side, head, expert) lists that call returns; after an sh_forward with bf16 storage only
 * what that pass's kernels needed - the source side alone, and for a k = 2 layer the tokens
 * of a head bucketed by their PAIR of selected experts instead of by expert.
 * Testing aid: lets a failing output be traced to the stage that produced it. */
int sh_debug_buffer(sh_layer* layer, int which, void** dev_ptr, size_t* bytes);

/* Reads the device status word (one blocking 4-byte copy on `stream`, which it drains).
 * 0 if every kernel so far completed normally, else the first SH_ERR_TIMEOUT / SH_ERR_BOUNDS
 * code recorded by a kernel that gave up a bounded wait or skipped a bad index. */
int sh_last_status(sh_layer* layer, void* stream);

/* The first 16 words of the device status block, copied to the HOST array words[16] (drains
 * `stream`): [0] the status word; [1..6] where the first bounded wait gave up - block, thread,
 * shared-memory address of the barrier, parity waited for, grid size, block size; [8..11] the
 * first failed index check of the debug library - site, value, limit, block. */
int sh_status_block(sh_layer* layer, int32_t* words, void* stream);

/* Clears the status block (asynchronously on `stream`): the status word, the diagnostics, and
 * the tile and grid-barrier counters that a kernel which gave up may have left half-way.  After
 * a non-zero sh_last_status, call this before the next sh_forward. */
int sh_clear_status(sh_layer* layer, void* stream);

/* Every sub-buffer of the workspace is followed by 256 guard bytes that sh_set_weights fills
 * with a pattern.  Checks them all (one small kernel; drains `stream`): SH_OK, or SH_ERR_BOUNDS
 * with the number of damaged words in sh_last_error() when some kernel wrote past the end of
 * its buffer.  A testing aid that costs nothing in sh_forward. */
int sh_check_guards(sh_layer* layer, void* stream);

/* Self-tests of the error paths; neither touches memory outside the status block.
 *   which = 0: a one-thread kernel waits, through the bounded wait every kernel of the library
 *              uses, on a barrier that nothing signals, with a limit of `arg` nanoseconds
 *              (at most 1e9).  It gives up, records SH_ERR_TIMEOUT and the diagnostics words, and
 *              returns; the context stays usable.  sh_clear_status afterwards.
 *   which = 1: (debug library only, else SH_ERR_UNSUPPORTED) runs the index check on the value
 *              `arg` against the limit 10; a value outside records SH_ERR_BOUNDS and its
 *              diagnostics.
 * Enqueues one kernel on `stream`. */
int sh_selftest(sh_layer* layer, int which, uint64_t arg, void* stream);

/* Output precision of sh_forward for a layer configured with bf16 storage (Sec. 2.2, the MoE output
 * equation is summed in fp32 on chip either way): enable != 0 makes every later sh_forward (and
 * sh_forward_stamped / sh_forward_timed) write `out` as IEEE fp16 [batch, seq_out, d_model] - each
 * fp32 result rounded once, to nearest even - instead of fp32; the buffer is then half the size and
 * must still be 16-byte aligned.  A host-fed caller halves its device-to-host bytes this way.
 * Host call, no launch.  SH_ERR_UNSUPPORTED for the fp32 configuration and the dense comparator;
 * sh_backward and the fp32 configuration always use fp32. */
int sh_set_output_f16(sh_layer* layer, int enable);

/* 1 if the library was built with -DSH_DEBUG: every token-list entry, tile-table field and expert
 * index read from memory is range-checked before it is used (a failed check records SH_ERR_BOUNDS
 * and the access is skipped), and launch-structure switches are read from the environment when the
 * weights are set (SH_NO_PDL, SH_NO_OVERLAP, SH_QK_ONE_GRID, SH_QK_SINGLE, SH_O_SINGLE,
 * SH_NO_PERSISTENT, SH_SORT_SEPARATE, SH_NO_FRONT, SH_ATTN_ADJACENT, SH_SIMT_STAGES: A/B and test aids).
 * 0 for the release library, which has neither. */
int sh_is_debug_build(void);

/* Number of kernel launches the last sh_forward enqueued. */
int sh_launch_count(const sh_layer* layer);

/* Reason for the last failure on this host thread ("" if none). */
const char* sh_last_error(void);

/* Free the handle (NULL is allowed).  Does not touch caller-owned device memory. */
void sh_destroy(sh_layer* layer);

#ifdef __cplusplus
}
#endif
#endif /* SWITCHHEAD_H_ */
