/*
 * bita.h - C ABI of the BiTA tree-decoding step for one NVIDIA B200 (sm_100a).
 *
 * One call of bita_step is one forward pass of the paper's streamlined generation
 * and verification (arXiv 2401.12522, Sec. 3.2, Appendix B, Algorithm 1, t > 1):
 * a packed block of rows - the last accepted token, the flattened draft-candidate
 * tree of the previous pass, and groups of learnable mask tokens - runs through a
 * frozen LLaMA-style decoder with tree-based attention over the KV cache; greedy
 * verification then keeps the longest root-to-node path whose tokens equal the
 * model's own argmax predictions, the mask tokens' top-k predictions fill the
 * next tree, and the cache entries of the accepted path are compacted in place.
 *
 * Conventions
 *   - Every pointer is tagged HOST or DEVICE below.  DEVICE memory (weights, KV
 *     cache, workspace) is allocated and owned by the caller; the library borrows
 *     it and allocates only small host-side structures and a few pinned host bytes.
 *   - All matrices are bf16, row-major [out_features][in_features].
 *   - Every call returns 0 (BITA_OK) or a negative BITA_ERR_* code.  Arguments are
 *     checked on the host before anything is launched.  Nothing throws or aborts.
 *   - Calls on one context are not thread-safe.  Work is enqueued on the stream
 *     given to bita_init.
 */
#ifndef BITA_H_
#define BITA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BITA_OK 0
#define BITA_ERR_INVALID_ARG (-1)   /* NULL pointer, non-positive or unsupported dimension          */
#define BITA_ERR_BAD_TEMPLATE (-2)  /* parent[i] >= i, rank or attach out of range, too many rows    */
#define BITA_ERR_KV_FULL (-3)       /* the pass would write beyond C_max                             */
#define BITA_ERR_WORKSPACE (-4)     /* workspace too small or misaligned                              */
#define BITA_ERR_CUDA (-5)          /* a CUDA runtime call failed; see bita_last_cuda_error           */
#define BITA_ERR_TIMEOUT (-6)       /* a bounded device-side wait ran out (status word set)           */
#define BITA_ERR_NOT_PREFILLED (-7) /* bita_step before bita_prefill                                  */
#define BITA_ERR_STATIC_SCRATCH (-8) /* problem needs more than the library's built-in scratch array  */

#define BITA_MAX_NODES 160          /* tree nodes, root excluded                                      */
#define BITA_MAX_ROWS 352           /* rows of the packed block: 1 + N + G * n_mask (a multiple of 32) */
#define BITA_MAX_DEPTH 16
#define BITA_MAX_TOPK 16            /* largest rank + 1 a template may use                            */
#define BITA_MAX_MASK 8             /* mask tokens per group                                          */
#define BITA_MAX_BATCH 16           /* sequences of one context; batch * rows per sequence <= BITA_MAX_ROWS */

/* Model dimensions (the paper only says "LLaMA-2", Sec. 4.1): RMSNorm, rotary
 * embedding with half-split pairing, SwiGLU, no biases, untied LM head. */
typedef struct {
  int32_t L;          /* decoder layers                                                         */
  int32_t d;          /* model width, multiple of 8                                             */
  int32_t H;          /* query heads                                                            */
  int32_t H_kv;       /* key/value heads, divides H                                             */
  int32_t D;          /* head dimension: 64 or 128                                              */
  int32_t F;          /* SwiGLU width, multiple of 8                                            */
  int32_t V;          /* vocabulary                                                             */
  int32_t P;          /* prompt (prefix) tokens per layer, 0..64 (paper default 16, Sec. 4.1)   */
  int32_t C_max;      /* capacity of the KV cache in tokens                                     */
  float rms_eps;
  float rope_theta;
} bita_model_dims;

/* Weights: DEVICE pointers to bf16 data, borrowed for the life of the context.
 * The arrays of per-layer pointers themselves are HOST arrays of length L. */
typedef struct {
  const void* tok_emb;              /* [V][d]                                                   */
  const void* mask_emb;             /* [n_mask][d]  learnable mask-token embeddings (Sec. 3.1)  */
  const void* g_final;              /* [d]                                                      */
  const void* lm_head;              /* [V][d]                                                   */
  const void* const* wqkv;          /* L x [(H + 2 H_kv) D][d]   rows: all q heads, k heads, v  */
  const void* const* wo;            /* L x [d][H D]                                             */
  const void* const* wg;            /* L x [F][d]                                               */
  const void* const* wu;            /* L x [F][d]                                               */
  const void* const* wd;            /* L x [d][F]                                               */
  const void* const* g_attn;        /* L x [d]                                                  */
  const void* const* g_ffn;         /* L x [d]                                                  */
  const void* const* prompt_k;      /* L x [H_kv][P][D]  deep prompt: per-layer key prefix,     */
  const void* const* prompt_v;      /* L x [H_kv][P][D]  seen by mask tokens only (Sec. 3.1)    */
} bita_weights;

/* Shape of the draft-candidate tree and of the mask groups (Sec. 3.2, Fig. 4).
 * Node i (flattened depth by depth, Appendix B) hangs under parent[i] (-1 = the last
 * accepted token) and is filled with the (rank[i]+1)-th best prediction of the mask
 * token of its depth.  attach[g] is the row a group of n_mask mask tokens follows:
 * -1 = the last accepted token, else a node.  G = N + 1 (one group per node and one
 * for the last token) is the paper's method (Algorithm 1); G = 1, attach = {-1} is
 * the single-group variant.  All arrays are HOST arrays, copied at init. */
typedef struct {
  int32_t N;
  const int32_t* parent;            /* N entries, -1 <= parent[i] < i                           */
  const int32_t* rank;              /* N entries, 0 <= rank[i] < BITA_MAX_TOPK                  */
  int32_t G;
  const int32_t* attach;            /* G entries, -1 <= attach[g] < N, all distinct             */
} bita_tree_template;

/* KV cache: DEVICE, bf16, layout [L][B][H_kv][C_max][D] for keys and for values, B = sequences
 * of the context (1 for bita_init: [L][H_kv][C_max][D]). */
typedef struct {
  void* k;
  void* v;
  int32_t C_max;
} bita_kv;

/* Result of one pass (HOST, caller-owned). */
typedef struct {
  int32_t status;                        /* 0, or BITA_ERR_TIMEOUT reported by the device        */
  int32_t n_out;                         /* tokens emitted = accepted drafts + 1                  */
  int32_t new_len;                       /* tokens in the cache after compaction                  */
  int32_t out_tokens[BITA_MAX_DEPTH + 1];
  int32_t accepted_idx[BITA_MAX_DEPTH];  /* node indices of the accepted path, root excluded      */
  int32_t next_tree[BITA_MAX_NODES];     /* tokens of the next pass's tree, -1 = node disabled    */
} bita_step_out;

typedef struct bita_ctx bita_ctx;

/* Bytes of DEVICE workspace bita_init needs for these dimensions (256-byte aligned). */
int bita_workspace_bytes(const bita_model_dims* dims, const bita_tree_template* tmpl, int n_mask,
                         size_t* out_bytes);

/* Create a context.  `workspace` is DEVICE memory of at least bita_workspace_bytes;
 * `cuda_stream` is a cudaStream_t (NULL = the legacy default stream).  The context
 * starts empty: call bita_prefill before bita_step. */
int bita_init(bita_ctx** out, const bita_model_dims* dims, const bita_weights* w,
              const bita_tree_template* tmpl, int n_mask, void* workspace, size_t workspace_bytes,
              void* cuda_stream);

/* First pass (Algorithm 1, t = 1; Appendix B): `count` HOST token ids are appended
 * to the cache (in chunks, causal attention), the last one's argmax becomes the
 * last accepted token, and the first tree is drafted by one mask group that follows
 * it.  `out` may be NULL; otherwise n_out = 1, out_tokens[0] = the emitted token. */
int bita_prefill(bita_ctx* ctx, bita_kv* kv, const int32_t* tokens, int32_t count, bita_step_out* out);

/* One pass for t > 1 (Algorithm 1, else-branch).  `tree_tokens` is a HOST array of N
 * token ids (-1 disables a node) or NULL to verify the tree the previous pass built.
 * Blocks until the result record is on the host.  Copies: N ints to the device,
 * the result record back. */
int bita_step(bita_ctx* ctx, bita_kv* kv, const int32_t* tree_tokens, bita_step_out* out);

/* The same pass with every input already on the device: `tree_tokens_dev` is a
 * DEVICE array of N ints or NULL.  Only enqueues work on the stream; nothing is
 * waited for.  bita_step_finish waits for the most recent pass and fills `out`. */
int bita_step_enqueue(bita_ctx* ctx, bita_kv* kv, const int32_t* tree_tokens_dev);
int bita_step_finish(bita_ctx* ctx, bita_step_out* out);

/* ---- several sequences in one pass ----
 * The paper measures one sequence at a time (Sec. 4.1, batch size 1); a weight-streaming pass costs
 * nearly the same for a few hundred rows as for 69, so the same pass can carry the blocks of
 * `batch` independent sequences: batch * (1 + N + G * n_mask) <= BITA_MAX_ROWS rows, sequence-major.
 * Each sequence has its own cache slab, length, last token, drafted tree, verification walk
 * (Algorithm 1, else-branch, once per sequence), accepted length and compaction; the sequences
 * share the tree template and the weights only.  bita_init_batch(.., batch = 1, ..) is bita_init.
 *   bita_prefill_seq        first pass of ONE sequence (0 <= seq < batch), as bita_prefill
 *   bita_step_batch         tree_tokens: HOST [batch][N] or NULL; out: HOST array of `batch` records
 *   bita_step_batch_enqueue tree_tokens_dev: DEVICE [batch][N] or NULL; only enqueues
 *   bita_step_batch_finish  waits, fills `batch` records; BITA_ERR_NOT_PREFILLED unless every sequence was prefilled
 *   bita_rewind_seq         bita_rewind for one sequence
 * bita_step / bita_step_enqueue / bita_step_finish / bita_prefill / bita_rewind act on sequence 0 and
 * return BITA_ERR_INVALID_ARG on a context of more than one sequence (the step calls). */
int bita_workspace_bytes_batch(const bita_model_dims* dims, const bita_tree_template* tmpl, int n_mask,
                               int32_t batch, size_t* out_bytes);
int bita_init_batch(bita_ctx** out, const bita_model_dims* dims, const bita_weights* w,
                    const bita_tree_template* tmpl, int n_mask, int32_t batch, void* workspace,
                    size_t workspace_bytes, void* cuda_stream);
int bita_prefill_seq(bita_ctx* ctx, bita_kv* kv, int32_t seq, const int32_t* tokens, int32_t count,
                     bita_step_out* out);
int bita_step_batch(bita_ctx* ctx, bita_kv* kv, const int32_t* tree_tokens, bita_step_out* out);
int bita_step_batch_enqueue(bita_ctx* ctx, bita_kv* kv, const int32_t* tree_tokens_dev);
int bita_step_batch_finish(bita_ctx* ctx, bita_step_out* out);
int bita_rewind_seq(bita_ctx* ctx, bita_kv* kv, int32_t seq, int32_t new_len, int32_t last_token);
/* Sequences of the context. */
int bita_batch(const bita_ctx* ctx);

/* Back to the state after bita_init: empty caches, no last tokens, no trees (all sequences). */
int bita_reset(bita_ctx* ctx, bita_kv* kv);

/* Cut the decoding state back (Algorithm 1 cuts the output at <EOS>; a caller that goes on after
 * such a cut, or that explored a continuation, needs the cache cut too): keep the first `new_len`
 * cache entries, make `last_token` the last accepted token and drop the drafted tree.
 * 0 <= new_len <= current length. */
int bita_rewind(bita_ctx* ctx, bita_kv* kv, int32_t new_len, int32_t last_token);

/* Debugging aid for parity checks: when `dev_buf` (DEVICE, fp32) is non-NULL every
 * later pass also stores the residual stream after each layer ([L][BITA_MAX_ROWS][d],
 * the first `rows` rows of each slab valid) and the logits ([rows][V]) there, rows =
 * rows of that pass.  NULL switches it off.
 * `bytes` must hold L * BITA_MAX_ROWS * d + BITA_MAX_ROWS * V floats. */
int bita_set_debug_buffer(bita_ctx* ctx, void* dev_buf, size_t bytes);

/* Read back what the most recent pass left for inspection (Algorithm 1 names the quantities: the
 * output logits L^t, and the top-k predictions of the mask tokens that form C^t), into HOST memory:
 *   BITA_DEBUG_LOGITS       fp32 [rows][V]     logits of every row of the pass
 *   BITA_DEBUG_TOPK         int32 [rows][BITA_MAX_TOPK]  selected token ids per row: slot 0 = argmax;
 *                           slots 1.. are filled for mask rows only, up to the template's k
 *   BITA_DEBUG_HIDDEN + l   fp32 [rows][d]     residual stream after decoder layer l
 * rows = rows of that pass.  Logits and hidden states need a debug buffer set BEFORE the pass
 * (bita_set_debug_buffer: the caller owns all device memory, so it provides the storage).  Waits
 * for the stream.  `bytes` = capacity of dst; BITA_ERR_INVALID_ARG when too small, when no pass
 * has run, or when the quantity was not recorded. */
#define BITA_DEBUG_LOGITS 1
#define BITA_DEBUG_TOPK 2
#define BITA_DEBUG_HIDDEN 1000
int bita_debug_fetch(bita_ctx* ctx, int what, void* dst, size_t bytes);

/* Bound of every device-side wait (mbarriers, split-K counters, cluster hand-overs) of later passes,
 * in nanoseconds; default 2 s.  A wait that runs out sets the context's status word: the pass
 * returns BITA_ERR_TIMEOUT, and so does every later one until bita_reset. */
int bita_set_wait_limit(bita_ctx* ctx, uint64_t limit_ns);

/* Self-check of that mechanism: runs one thread through the library's bounded wait on a barrier
 * nobody arrives on, with the given limit (1 us .. 1 s).  The wait must give up, so the expected
 * return value is BITA_ERR_TIMEOUT, and the context's status word is set as after a real timeout
 * (clear it with bita_reset).  Returns 0 if the wait did not report, which would be a defect. */
int bita_probe_wait_timeout(bita_ctx* ctx, uint64_t limit_ns);

/* Per-kernel-family device timing of later passes, for roofline reports.  When on, a pass records
 * a CUDA event on the context's stream wherever the kernel family changes, so that every run of
 * consecutive launches of one family (e.g. O, gate/up, down and the next layer's q/k/v projection)
 * is timed as a whole, overlapping as it does in an untimed pass.
 * bita_get_kernel_timing waits for the stream and returns, for the most recent pass, the summed
 * milliseconds and launch counts per family into HOST arrays of BITA_TIMING_FAMILIES entries:
 * [0] projections (QKV, O, gate/up, down, LM head), [1] tree attention. */
#define BITA_TIMING_FAMILIES 2
int bita_set_kernel_timing(bita_ctx* ctx, int on);
int bita_get_kernel_timing(bita_ctx* ctx, float* ms, int32_t* launches);

/* Rows one sequence contributes to the packed block of a step (1 + N + G * n_mask). */
int bita_block_rows(const bita_ctx* ctx);
/* Number of kernel launches the most recent bita_step / bita_step_enqueue / bita_prefill made. */
int bita_last_launch_count(const bita_ctx* ctx);

void bita_destroy(bita_ctx* ctx);
const char* bita_strerror(int code);
/* Last cudaError_t seen by a failing call on this thread (0 if none). */
int bita_last_cuda_error(void);

/* ---- single operators of the step, exported for per-kernel parity and timing ---- */

/* Y[m][n] = sum_k X[m][k] * W[n][k]  (the small-M weight-streaming projection of the
 * decoder; Sec. 3.2, last paragraph: the pass is bound by memory traffic, not arithmetic).  X: DEVICE bf16 [M][K],
 * W: DEVICE bf16 [N][K], Y: DEVICE fp32 [M][N].  1 <= M <= BITA_MAX_ROWS, K % 8 == 0.
 * `workspace` DEVICE scratch of bita_gemm_workspace_bytes(M, N, K), 256-byte aligned. */
int bita_gemm_workspace_bytes(int32_t M, int32_t N, int32_t K, size_t* out_bytes);
int bita_gemm_bf16(const void* X, const void* W, void* Y, int32_t M, int32_t N, int32_t K,
                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Tree-based attention (Sec. 3.2, Fig. 6) for B independent sequences.
 *   q      DEVICE bf16 [B][M][H][D]   (already rotated)
 *   k, v   DEVICE bf16 [B][H_kv][C_max][D]; slots [0, C) are the context every row
 *          sees, slots [C, C+M) hold the block's own rows
 *   vis    DEVICE uint32 [B][M][ceil(M/32)]: bit j of row r set iff row r may see block row j
 *   prompt_k/v  DEVICE bf16 [H_kv][P][D] or NULL; sees_prompt DEVICE uint8 [B][M] or NULL
 *   ctx_len     DEVICE int32 [B]: C per sequence, C + M <= C_max
 *   out    DEVICE bf16 [B][M][H*D]
 * `workspace` DEVICE scratch of bita_attention_workspace_bytes, 256-byte aligned: room for the
 * partial results of the key slices; 0 bytes (workspace may be NULL) when the launch takes a
 * single key slice.  (The slices normally run as one thread-block cluster and merge on chip; the
 * scratch is written when that launch form is refused, or when bita_set_attention_route(1) asks
 * for it, and a second kernel merges.)  A wait between key slices that runs out (2 s) leaves
 * wrong output rather than a hang. */
int bita_attention_workspace_bytes(int32_t B, int32_t M, int32_t H, int32_t D, size_t* out_bytes);
/* The same for a cache of capacity C_max, never less than the above.  With a long cache (16384 keys and
 * more) and a workspace of this size, bita_tree_attention may cut the keys into as many slices (up to
 * 64) as make the waves of CTAs come out even - e.g. 8 sequences x 32 heads are 256 CTAs, two uneven
 * waves on 148 SMs, but 1024 CTAs of a quarter of the keys each are seven even ones - and merges the
 * slices' partial results with its second kernel.  With the smaller workspace the call still works,
 * with the cluster shape. */
int bita_attention_workspace_bytes_long(int32_t B, int32_t M, int32_t H, int32_t D, int32_t C_max,
                                        size_t* out_bytes);
/* Diagnostic, process-wide: 0 (default) = key slices merge inside a thread-block cluster whenever
 * that launch form is accepted; 1 = always through the workspace and the separate merge kernel.
 * Affects bita_tree_attention and the passes of every context. */
int bita_set_attention_route(int route);
int bita_tree_attention(const void* q, const void* k, const void* v, const uint32_t* vis,
                        const void* prompt_k, const void* prompt_v, const uint8_t* sees_prompt,
                        const int32_t* ctx_len, void* out, int32_t B, int32_t M, int32_t H,
                        int32_t H_kv, int32_t D, int32_t P, int32_t C_max, void* workspace,
                        size_t workspace_bytes, void* cuda_stream);

/* Tree attention for callers that must not allocate device memory.  (The paper has no counterpart:
 * this is a convenience of the library, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a serving loop whose memory pool
 * was sized once and frozen, a plug-in that lives inside another framework's allocator, a latency
 * path that cannot afford the device-wide synchronisation an allocation implies.  Such a caller
 * can hold q, k, v and out, but has nowhere to get the split-KV scratch that bita_tree_attention
 * asks for.  This variant takes the same arguments minus the workspace and keeps its scratch in a
 * fixed array inside the library's device image: BITA_STATIC_SCRATCH_BYTES per GPU, resident on
 * every GPU that loads the library, until the process exits.
 *
 * Limits and rules
 *   - The scratch needed is what bita_attention_workspace_bytes reports for (B, M, H, D).  If that
 *     exceeds BITA_STATIC_SCRATCH_BYTES the call returns BITA_ERR_STATIC_SCRATCH and launches
 *     nothing.  (7B-shaped steps, H = 32, M = 69, D = 128, B = 1, need 4.6 MB and fit; 133 rows
 *     at that head count do not.  Launches with so many (sequence, head) pairs that each takes a
 *     single key slice need no scratch and are always accepted.)
 *   - With more than one key slice this entry always takes the workspace route: the slices write
 *     their partial results into the array and a merge kernel reads them back (two launches).
 *   - The first call on each device looks up the array's device address (one runtime query, no
 *     allocation).  Make that first call outside any stream capture.
 *   - The call itself allocates nothing: no cudaMalloc, no cudaFree, no allocating library call.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left.
 *     That is harmless here, because each call overwrites every slot it later reads, but two
 *     calls whose kernels overlap on the GPU (different streams, no ordering) race on it: order
 *     them on one stream or with events.
 * Results are the same as bita_tree_attention's. */
#define BITA_STATIC_SCRATCH_BYTES (8u << 20)
int bita_tree_attention_static(const void* q, const void* k, const void* v, const uint32_t* vis,
                               const void* prompt_k, const void* prompt_v, const uint8_t* sees_prompt,
                               const int32_t* ctx_len, void* out, int32_t B, int32_t M, int32_t H,
                               int32_t H_kv, int32_t D, int32_t P, int32_t C_max, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* BITA_H_ */
