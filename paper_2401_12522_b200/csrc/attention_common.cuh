// Tree-based attention (Sec. 3.2, Fig. 6): arguments, partial-result format and merge of key slices.
//
// Keys of one (sequence, kv head): cache slots [0, C) are the context every row sees, slots
// [C, C+M) are the block's own rows (seen according to the ancestor bitmask), and the layer's P
// prompt-prefix keys (a separate buffer) are seen by mask rows only (Sec. 3.1).  The key sequence
// is cut into S slices, one CTA each; a slice leaves, per query row, its running maximum (log2
// domain), its running sum and its unnormalised output.  The slices of a row are merged in slice
// order: inside the attention kernel when all its CTAs are resident together (`sync` given: each
// slice merges an equal share of its row tile's rows once all slices of the tile have arrived),
// else by k_attn_merge.  A single slice writes the output itself.
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
  const int32_t* ctx_len;    // [B]
  int32_t vis_batch_stride;  // words between sequences (0 = shared)
  int32_t sp_batch_stride;
  bf16* out;                 // [B][M][H*D]
  float* part_ml;            // [B][H][S][M][2]  (running max in log2 units, running sum)
  float* part_acc;           // [B][H][S][M][D]
  int32_t B, M, W, H, H_kv, D, P, C_max, S;
  int32_t row_tiles;         // ceil(M / 128): query rows per CTA
  float scale_log2;          // log2(e) / sqrt(D)
  int32_t* sync;             // in-kernel merge: [2][B*H*row_tiles] arrival / departure counters, zero
                             // before the launch and left zero; null = partial results only
  int32_t* status;           // sticky error word for a wait that ran out (may be null)
};

// Partial results of one row (all its slices), loaded first so that several rows' loads fly together.
template <int D>
struct MergeRow {
  float ms[8], ls[8], v[8][D / 32];
};

template <int D>
__device__ __forceinline__ void attn_merge_load(const AttnArgs& a, int b, int h, int gr, int lane, MergeRow<D>& m) {
  constexpr int VW = D / 32;
  const size_t p0 = (((size_t)b * a.H + h) * a.S) * a.M + gr;
#pragma unroll
  for (int s = 0; s < 8; ++s) {
    m.ms[s] = -INFINITY;
    m.ls[s] = 0.f;
#pragma unroll
    for (int e = 0; e < VW; ++e) m.v[s][e] = 0.f;
    if (s < a.S) {
      const size_t pi = p0 + (size_t)s * a.M;
      const float2 ml = __ldcg(reinterpret_cast<const float2*>(a.part_ml + pi * 2));
      m.ms[s] = ml.x;
      m.ls[s] = ml.y;
      if constexpr (VW == 4) {
        const float4 t = __ldcg(reinterpret_cast<const float4*>(a.part_acc + pi * D) + lane);
        m.v[s][0] = t.x; m.v[s][1] = t.y; m.v[s][2] = t.z; m.v[s][3] = t.w;
      } else {
        const float2 t = __ldcg(reinterpret_cast<const float2*>(a.part_acc + pi * D) + lane);
        m.v[s][0] = t.x; m.v[s][1] = t.y;
      }
    }
  }
}

// Merged, normalised output of one row (slice order).  `lane` owns D / 32 consecutive features.
template <int D>
__device__ __forceinline__ void attn_merge_finish(const AttnArgs& a, int b, int h, int gr, int lane, const MergeRow<D>& m) {
  constexpr int VW = D / 32;
  float mx = -INFINITY;
#pragma unroll
  for (int s = 0; s < 8; ++s) mx = fmaxf(mx, m.ms[s]);
  float l = 0.f, o[VW];
#pragma unroll
  for (int e = 0; e < VW; ++e) o[e] = 0.f;
#pragma unroll
  for (int s = 0; s < 8; ++s) {
    if (m.ms[s] == -INFINITY) continue;
    const float w = exp2f(m.ms[s] - mx);
    l += m.ls[s] * w;
#pragma unroll
    for (int e = 0; e < VW; ++e) o[e] += m.v[s][e] * w;
  }
  const float inv = l > 0.f ? 1.0f / l : 0.f;
  bf16* dst = a.out + (((size_t)b * a.M + gr) * a.H + h) * D + lane * VW;
#pragma unroll
  for (int e = 0; e < VW; e += 2)
    *reinterpret_cast<__nv_bfloat162*>(dst + e) = __floats2bfloat162_rn(o[e] * inv, o[e + 1] * inv);
}

// Rows [r_lo, r_hi) of a row tile merged by `nwarps` warps, three rows per warp in flight.
template <int D>
__device__ __forceinline__ void attn_merge_rows(const AttnArgs& a, int b, int h, int row0, int r_lo, int r_hi, int warp,
                                                int nwarps, int lane) {
  for (int r = r_lo + warp; r < r_hi; r += 3 * nwarps) {
    MergeRow<D> m0, m1, m2;
    const int r1 = r + nwarps, r2 = r + 2 * nwarps;
    attn_merge_load<D>(a, b, h, row0 + r, lane, m0);
    if (r1 < r_hi) attn_merge_load<D>(a, b, h, row0 + r1, lane, m1);
    if (r2 < r_hi) attn_merge_load<D>(a, b, h, row0 + r2, lane, m2);
    attn_merge_finish<D>(a, b, h, row0 + r, lane, m0);
    if (r1 < r_hi) attn_merge_finish<D>(a, b, h, row0 + r1, lane, m1);
    if (r2 < r_hi) attn_merge_finish<D>(a, b, h, row0 + r2, lane, m2);
  }
}

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
