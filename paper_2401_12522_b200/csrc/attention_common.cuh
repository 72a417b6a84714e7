// Tree-based attention (Sec. 3.2, Fig. 6): arguments, partial-result format and merge of key slices.
//
// Keys of one (sequence, kv head): cache slots [0, C) are the context every row sees, slots
// [C, C+M) are the block's own rows (seen according to the ancestor bitmask), and the layer's P
// prompt-prefix keys (a separate buffer) are seen by mask rows only (Sec. 3.1).  The key sequence
// is cut into S slices, one CTA each; a slice leaves, per query row, its running maximum (log2
// domain), its running sum and its unnormalised output.  The slices of a row are merged in slice
// order: inside the attention kernel when the slices are launched as one thread-block cluster
// (each slice merges an equal share of its row tile's rows), else by k_attn_merge from partial
// results in global memory.  A single slice writes the output itself.
#pragma once

#include "common.cuh"

namespace bita {

struct AttnArgs {
  const bf16* q;             // [B][M][H][D]
  const bf16* k;             // [B][H_kv][C_max][D]
  const bf16* v;
  const uint32_t* vis;       // [B][M][W]
  const bf16* prompt_k;      // [H_kv][P][D] or null
  const bf16* prompt_v;
  const uint8_t* sees_prompt;  // [B][M] or null
  const int32_t* ctx_len;    // C of sequence b at ctx_len[b * ctx_len_stride]
  int32_t ctx_len_stride;
  int32_t vis_batch_stride;  // words between sequences (0 = shared)
  int32_t sp_batch_stride;
  bf16* out;                 // [B][M][H*D]
  float* part_ml;            // [B][H][S][M][2]  (running max in log2 units, running sum)
  float* part_acc;           // [B][H][S][M][D]
  int32_t B, M, W, H, H_kv, D, P, C_max, S;
  int32_t row_tiles;         // ceil(M / 128): query rows per CTA
  float scale_log2;          // log2(e) / sqrt(D)
  int32_t cluster;           // 1: the S slices of a (sequence, head, row tile) form a thread-block cluster
                             // and merge through distributed shared memory; 0: they leave partial
                             // results in part_ml / part_acc for k_attn_merge
  int32_t* status;           // sticky error word for a wait that ran out (may be null)
  unsigned long long wait_ns;  // bound of every device-side wait of the launch
};

// Merge the S slices of each (sequence, head, row) in slice order; write bf16 [B][M][H*D].
// grid = (M, H, B), D / 2 threads (one float2 of the output each).
template <int D>
__global__ void k_attn_merge(AttnArgs a) {
  pdl_launch();
  pdl_wait();
  const int r = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const size_t p0 = (((size_t)b * a.H + h) * a.S) * a.M + r;
  float mx = -INFINITY;
  for (int s = 0; s < a.S; ++s) mx = fmaxf(mx, a.part_ml[(p0 + (size_t)s * a.M) * 2]);
  float l = 0.f;
  float2 o = make_float2(0.f, 0.f);
  const int c = threadIdx.x * 2;
  for (int s = 0; s < a.S; ++s) {
    const size_t pi = p0 + (size_t)s * a.M;
    const float ms = a.part_ml[pi * 2];
    if (ms == -INFINITY) continue;
    const float w = exp2f(ms - mx);
    l += a.part_ml[pi * 2 + 1] * w;
    const float2 v = *reinterpret_cast<const float2*>(a.part_acc + pi * D + c);
    o.x += v.x * w;
    o.y += v.y * w;
  }
  const float inv = l > 0.f ? 1.0f / l : 0.f;
  *reinterpret_cast<__nv_bfloat162*>(a.out + (((size_t)b * a.M + r) * a.H + h) * D + c) =
      __floats2bfloat162_rn(o.x * inv, o.y * inv);
}

}  // namespace bita
