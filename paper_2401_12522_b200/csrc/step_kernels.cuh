// Element-wise and integer kernels of one decoding pass: embedding/packing, argmax/top-k
// selection, the greedy verification walk, next-tree construction and cache compaction.
// (Residual add, RMSNorm, rotary embedding, the cache write and SwiGLU live in the projection
// epilogues.)
// Every kernel starts with the programmatic-dependent-launch pair: release the next kernel's
// prologue, then wait for the predecessors before touching memory.
#pragma once

#include "common.cuh"
#include "gemm_tc.cuh"

namespace bita {

// ---------------------------------------------------------------------------------------------
// Packing (Sec. 3.2, Appendix B: the candidate tree and its mask groups become one row sequence):
// row 0 = last accepted token, rows 1..N = tree tokens (token -1 -> zero row), then the mask
// embeddings.  Position ids: C + rel_pos.
// x: fp32 [B * M][d] residual stream; pos: int32 [B * M].  `states`: the context's per-sequence
// states; `tree_tokens`: [B][N] or null (each sequence's own drafted tree).
__global__ void k_embed(DevPlan plan, const DevState* __restrict__ states, const int32_t* __restrict__ tree_tokens,
                        const int32_t* __restrict__ query_tokens, const bf16* __restrict__ tok_emb,
                        const bf16* __restrict__ mask_emb, int d, int V, float* __restrict__ x,
                        int32_t* __restrict__ pos, int32_t* __restrict__ row_token,
                        const float2* __restrict__ rope_tab, int half, float2* __restrict__ rope_blk,
                        const bf16* __restrict__ gain0, bf16* __restrict__ xhat,
                        unsigned long long* __restrict__ sumsq, int n_slots) {
  pdl_launch();
  pdl_wait();
  const int r = blockIdx.x;                              // global row
  const int b = r / plan.M, rs = r - b * plan.M;         // sequence of the block, row within it
  const DevState* st = states + plan.seq0 + b;
  const int kind = plan.row_kind[rs];
  const int idx = plan.row_idx[rs];
  const bf16* src = nullptr;
  int tok = -1;
  if (kind == ROW_ROOT) tok = st->root;
  else if (kind == ROW_NODE) tok = tree_tokens ? tree_tokens[(size_t)b * plan.N + idx] : st->tree[idx];
  else if (kind == ROW_QUERY) tok = query_tokens[idx];
  if (kind == ROW_MASK) src = mask_emb + (size_t)idx * d;
  else if (tok >= 0 && tok < V) src = tok_emb + (size_t)tok * d;
  if (threadIdx.x == 0) {
    pos[r] = st->len + plan.rel_pos[rs];
    row_token[r] = (tok >= 0 && tok < V) ? tok : -1;
  }
  float* xr = x + (size_t)r * d;
  bf16* hr = xhat + (size_t)r * d;
  float ss = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    const float v = src ? bf2f(src[c]) : 0.0f;
    xr[c] = v;
    hr[c] = f2bf(v * bf2f(gain0[c]));                     // input of the first projection: x * gain, unnormalised
    ss += v * v;
  }
  // RMSNorm statistics: slot 0 is this row's sum of squares, the later slots are accumulated by
  // the projections of the pass and start from zero
  __shared__ float red[32];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
    sumsq[r] = sumsq_to_fixed(t);
  }
  for (int sl = 1 + threadIdx.x; sl < n_slots; sl += blockDim.x) sumsq[(size_t)sl * BITA_MAX_ROWS + r] = 0ull;
  // (cos, sin) row of this row's position id, for the rotary embedding in the q/k/v projection
  const int p = st->len + plan.rel_pos[rs];
  for (int j = threadIdx.x; j < half; j += blockDim.x) rope_blk[(size_t)r * half + j] = rope_tab[(size_t)p * half + j];
}

// ---------------------------------------------------------------------------------------------
// Second half of the selection that starts in the LM head's epilogue (Algorithm 1: the argmax `a`
// of a token row, the top k predictions of a mask row): every tile of 128 vocabulary entries has
// left its best entries of each row as ordered keys; one block per row picks the overall best
// k of them, again one at a time ("the largest key below the previous pick").
// cand: [rows][tiles][BITA_MAX_TOPK]; sel_id, sel_val: [rows][BITA_MAX_TOPK], best first.
__global__ void __launch_bounds__(256) k_select_merge(DevPlan plan, const unsigned long long* __restrict__ cand, int tiles,
                                                      int32_t* __restrict__ sel_id, float* __restrict__ sel_val) {
  pdl_launch();
  pdl_wait();
  __shared__ unsigned long long red[8];
  __shared__ unsigned long long pick;
  const int r = blockIdx.x;                              // global row
  const int K = plan.row_kind[r % plan.M] == ROW_MASK ? plan.k_max : 1;
  const unsigned long long* row = cand + (size_t)r * tiles * BITA_MAX_TOPK;
  const int n = tiles * K;                           // entry e: tile e / K, slot e % K
  unsigned long long prev = ~0ull;
  for (int t = 0; t < K; ++t) {
    unsigned long long best = 0ull;
    for (int e = threadIdx.x; e < n; e += blockDim.x) {
      const unsigned long long k = row[(size_t)(e / K) * BITA_MAX_TOPK + (e % K)];
      if (k < prev && k > best) best = k;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned long long b = 0ull;
      for (int w = 0; w < (int)(blockDim.x >> 5); ++w) b = max(b, red[w]);
      pick = b;
      const bool none = (b >> 32) == 0ull;            // nothing left (or only NaN entries)
      sel_id[(size_t)r * BITA_MAX_TOPK + t] = none ? -1 : select_key_id(b);
      sel_val[(size_t)r * BITA_MAX_TOPK + t] = none ? -INFINITY : select_key_value(b);
    }
    __syncthreads();
    prev = pick;
    if ((prev >> 32) == 0ull) break;
  }
}

// ---------------------------------------------------------------------------------------------
// Greedy verification (Algorithm 1, else-branch, general-tree form) and next-tree construction
// (Algorithm 1, last step of the else-branch: the next candidates are the top-k picks of the mask
// group that hangs on the last accepted node).  One warp per sequence of the block (grid = B): lanes
// scan the children of the current node.  Sequences accept independently: each has its own tree
// tokens, walk, accepted length and next tree.
__global__ void k_accept(DevPlan plan, DevState* __restrict__ states, const int32_t* __restrict__ row_token_all,
                         const int32_t* __restrict__ sel_id_all, DevRecord* __restrict__ recs) {
  pdl_launch();
  pdl_wait();
  const int lane = threadIdx.x;
  const int N = plan.N;
  const int b = blockIdx.x;
  DevState* st = states + plan.seq0 + b;
  DevRecord* rec = recs + plan.seq0 + b;
  const int32_t* row_token = row_token_all + (size_t)b * plan.M;
  const int32_t* sel_id = sel_id_all + (size_t)b * plan.M * BITA_MAX_TOPK;
  int cur = -1;
  int a = sel_id[0];
  int n_acc = 0;
  for (int round = 0; round < BITA_MAX_DEPTH; ++round) {
    int found = 0x7fffffff;
    for (int x = lane; x < N; x += 32) {
      const int tok = row_token[1 + x];
      if (plan.parent[x] == cur && tok >= 0 && tok == a) { found = x; break; }   // lowest index first
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) found = min(found, __shfl_xor_sync(0xffffffffu, found, o));
    if (found == 0x7fffffff) break;
    if (lane == 0) { rec->accepted_idx[n_acc] = found; rec->out_tokens[n_acc] = a; }
    ++n_acc;
    cur = found;
    a = sel_id[(size_t)(1 + cur) * BITA_MAX_TOPK];
  }
  // group attached to the last accepted node, else to its nearest ancestor that has one
  int at = cur, shift = 0, g = -1;
  while (true) {
    g = plan.group_of[at + 1];
    if (g >= 0 || at < 0) break;
    at = plan.parent[at];
    ++shift;
  }
  const int C = st->len;
  __syncwarp();
  for (int x = lane; x < N; x += 32) {
    const int m = plan.depth[x] - 1 + shift;
    int tok = -1;
    if (g >= 0 && m < plan.n_mask) {
      const int mrow = 1 + N + g * plan.n_mask + m;
      tok = sel_id[(size_t)mrow * BITA_MAX_TOPK + plan.rank[x]];
    }
    rec->next_tree[x] = tok;
    st->tree[x] = tok;
  }
  for (int x = N + lane; x < BITA_MAX_NODES; x += 32) rec->next_tree[x] = -1;
  if (lane == 0) {
    rec->out_tokens[n_acc] = a;
    for (int j = n_acc + 1; j <= BITA_MAX_DEPTH; ++j) rec->out_tokens[j] = -1;
    for (int j = n_acc; j < BITA_MAX_DEPTH; ++j) rec->accepted_idx[j] = -1;
    rec->n_out = n_acc + 1;
    rec->n_acc = n_acc;
    rec->old_len = C;
    rec->new_len = C + 1 + n_acc;
    rec->status = states[0].status;                     // the context's one sticky status word
    st->len = C + 1 + n_acc;
    st->root = a;
  }
}

// First pass (Algorithm 1, t = 1): the last query row's argmax is emitted, the one mask group that
// follows it drafts the first tree.  `last` = this is the final chunk of the query.
__global__ void k_prefill_finish(DevPlan chunk, DevPlan step_plan, DevState* __restrict__ states,
                                 const int32_t* __restrict__ sel_id, DevRecord* __restrict__ recs, int last) {
  pdl_launch();
  pdl_wait();
  const int lane = threadIdx.x;
  DevState* st = states + chunk.seq0;                    // the first pass takes one sequence at a time
  DevRecord* rec = recs + chunk.seq0;
  const int C = st->len;
  const int T = chunk.n_query;
  __syncwarp();
  if (last) {
    const int a = sel_id[(size_t)(T - 1) * BITA_MAX_TOPK];
    const int N = step_plan.N;
    for (int x = lane; x < N; x += 32) {
      const int m = step_plan.depth[x] - 1;
      int tok = -1;
      if (m < chunk.n_mask) tok = sel_id[(size_t)(T + m) * BITA_MAX_TOPK + step_plan.rank[x]];
      rec->next_tree[x] = tok;
      st->tree[x] = tok;
    }
    for (int x = N + lane; x < BITA_MAX_NODES; x += 32) rec->next_tree[x] = -1;
    if (lane == 0) {
      rec->out_tokens[0] = a;
      for (int j = 1; j <= BITA_MAX_DEPTH; ++j) rec->out_tokens[j] = -1;
      for (int j = 0; j < BITA_MAX_DEPTH; ++j) rec->accepted_idx[j] = -1;
      rec->n_out = 1;
      rec->n_acc = 0;
      rec->old_len = C;
      rec->new_len = C + T;
      rec->status = states[0].status;
      st->root = a;
    }
  }
  if (lane == 0) st->len = C + T;
}

// ---------------------------------------------------------------------------------------------
// Cache compaction (Fig. 3 caption: rejected drafts and what follows them leave no trace): the
// j-th accepted node's entry moves from slot C+1+idx_j to slot C+1+j.  One thread
// owns a 16-byte column chunk and walks j upwards, which is alias-safe because idx_j >= j and
// idx is increasing along a path.  grid = (L * H_kv, B), cache layout [L][B][H_kv][C_max][D]: every
// sequence moves its own accepted entries (a different number per sequence) inside its own slabs.
__global__ void k_compact(const DevRecord* __restrict__ recs, int D, int C_max, int H_kv, int B, bf16* __restrict__ kc,
                          bf16* __restrict__ vc) {
  pdl_launch();
  pdl_wait();
  const DevRecord* rec = recs + blockIdx.y;
  const int n_acc = rec->n_acc;
  if (n_acc == 0) return;
  const int C = rec->old_len;
  const int chunks = D / 8;                       // 16-byte chunks per row
  const int l = blockIdx.x / H_kv, h = blockIdx.x - l * H_kv;
  const size_t base = (((size_t)l * B + blockIdx.y) * H_kv + h) * C_max * D;
  for (int t = threadIdx.x; t < 2 * chunks; t += blockDim.x) {
    bf16* buf = (t < chunks ? kc : vc) + base;
    const int c = (t < chunks ? t : t - chunks) * 8;
    for (int j = 0; j < n_acc; ++j) {
      const int src = C + 1 + rec->accepted_idx[j];
      const int dst = C + 1 + j;
      if (src != dst && src < C_max) {
        const uint4 v = *reinterpret_cast<const uint4*>(buf + (size_t)src * D + c);
        *reinterpret_cast<uint4*>(buf + (size_t)dst * D + c) = v;
      }
    }
  }
}

// Diagnostic: one thread runs the library's bounded mbarrier wait on a barrier that nobody ever
// arrives on, so the wait must run out after `limit_ns`, raise the status word and return.
__global__ void k_wait_probe(int32_t* __restrict__ status, unsigned long long limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, status, limit_ns);
}

__global__ void k_set_state(DevState* st, int len, int root) {   // st: the state of ONE sequence
  pdl_launch();
  pdl_wait();
  if (threadIdx.x == 0) { st->len = len; st->root = root; }
  for (int x = threadIdx.x; x < BITA_MAX_NODES; x += blockDim.x) st->tree[x] = -1;
}

__global__ void k_reset_state(DevState* states) {                 // grid = sequences of the context
  pdl_launch();
  pdl_wait();
  DevState* st = states + blockIdx.x;
  if (threadIdx.x == 0) { st->len = 0; st->root = -1; st->status = 0; st->pad = 0; }
  for (int x = threadIdx.x; x < BITA_MAX_NODES; x += blockDim.x) st->tree[x] = -1;
}

}  // namespace bita
