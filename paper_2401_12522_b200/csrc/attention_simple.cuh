// Tree-based attention (Sec. 3.2, Fig. 6), split over the key sequence, CUDA-core version.
//
// Virtual key sequence of one (sequence, kv head): [0, C) cached context (seen by every row),
// [C, C+M) the block's own rows (seen according to the visibility bitmask), [C+M, C+M+P) the
// layer's prompt prefix (seen by mask rows only, Sec. 3.1).  Each block handles one query head and
// one slice of that sequence, one warp per query row, lanes over keys for the scores and over
// head dimensions for the weighted sum; slices are merged by k_attn_merge in slice order.
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
  float* part_ml;            // [B][H][S][M][2]
  float* part_acc;           // [B][H][S][M][D]
  int32_t B, M, W, H, H_kv, D, P, C_max, S;
  float scale;
};

template <int D>
__global__ void __launch_bounds__(128) k_attn_simple(AttnArgs a) {
  constexpr int EPL = D / 32;                      // output dims per lane
  const int h = blockIdx.x, s = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kvh = h / (a.H / a.H_kv);
  const int C = a.ctx_len[b];
  const int total = C + a.M + a.P;
  int per = (total + a.S - 1) / a.S;
  per = (per + 31) & ~31;
  const int k0 = s * per, k1 = min(total, k0 + per);
  const bf16* kb = a.k + ((size_t)b * a.H_kv + kvh) * (size_t)a.C_max * D;
  const bf16* vb = a.v + ((size_t)b * a.H_kv + kvh) * (size_t)a.C_max * D;
  const bf16* pk = a.prompt_k ? a.prompt_k + (size_t)kvh * a.P * D : nullptr;
  const bf16* pv = a.prompt_v ? a.prompt_v + (size_t)kvh * a.P * D : nullptr;
  __shared__ float qs[4][D];

  for (int r = warp; r < a.M; r += 4) {
    const bf16* qr = a.q + (((size_t)b * a.M + r) * a.H + h) * D;
    __syncwarp();
    for (int c = lane; c < D; c += 32) qs[warp][c] = bf2f(qr[c]) * a.scale;
    __syncwarp();
    const uint32_t* visr = a.vis + (size_t)b * a.vis_batch_stride + (size_t)r * a.W;
    const bool sp = pk && pv && a.sees_prompt && a.P > 0 && a.sees_prompt[(size_t)b * a.sp_batch_stride + r];
    float m = -INFINITY, l = 0.f;
    float acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    for (int base = k0; base < k1; base += 32) {
      const int key = base + lane;
      bool ok = key < k1;
      const bf16* krow = nullptr;
      if (ok) {
        if (key < C) krow = kb + (size_t)key * D;
        else if (key < C + a.M) {
          const int j = key - C;
          ok = (visr[j >> 5] >> (j & 31)) & 1u;
          krow = kb + (size_t)key * D;
        } else {
          ok = sp;
          krow = pk + (size_t)(key - C - a.M) * D;
        }
      }
      float sc = -INFINITY;
      if (ok) {
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < D; c += 8) {
          const uint4 u = *reinterpret_cast<const uint4*>(krow + c);
          const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(p2[e]);
            dot = fmaf(qs[warp][c + 2 * e], f.x, dot);
            dot = fmaf(qs[warp][c + 2 * e + 1], f.y, dot);
          }
        }
        sc = dot;
      }
      const float cm = warp_max(sc);
      if (cm == -INFINITY) continue;                 // nothing visible in this group of 32 keys
      const float mn = fmaxf(m, cm);
      const float corr = (m == -INFINITY) ? 0.f : __expf(m - mn);
      const float p = ok ? __expf(sc - mn) : 0.f;
      l = l * corr + warp_sum(p);
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] *= corr;
      m = mn;
      const unsigned live = __ballot_sync(0xffffffffu, ok);
      for (int j = 0; j < 32; ++j) {
        if (!((live >> j) & 1u)) continue;
        const float pj = __shfl_sync(0xffffffffu, p, j);
        const int kj = base + j;
        const bf16* vrow = (kj < C + a.M) ? vb + (size_t)kj * D : pv + (size_t)(kj - C - a.M) * D;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = fmaf(pj, bf2f(vrow[lane + 32 * e]), acc[e]);
      }
    }
    const size_t pidx = (((size_t)b * a.H + h) * a.S + s) * a.M + r;
    if (lane == 0) { a.part_ml[pidx * 2] = m; a.part_ml[pidx * 2 + 1] = l; }
#pragma unroll
    for (int e = 0; e < EPL; ++e) a.part_acc[pidx * D + lane + 32 * e] = acc[e];
  }
}

// Merge the S slices of each (sequence, head, row) in slice order; write bf16 [B][M][H*D].
template <int D>
__global__ void k_attn_merge(AttnArgs a) {
  const int r = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const size_t p0 = (((size_t)b * a.H + h) * a.S) * a.M + r;
  float mx = -INFINITY;
  for (int s = 0; s < a.S; ++s) mx = fmaxf(mx, a.part_ml[(p0 + (size_t)s * a.M) * 2]);
  float l = 0.f;
  for (int s = 0; s < a.S; ++s) {
    const float ms = a.part_ml[(p0 + (size_t)s * a.M) * 2];
    if (ms != -INFINITY) l += a.part_ml[(p0 + (size_t)s * a.M) * 2 + 1] * __expf(ms - mx);
  }
  const float inv = l > 0.f ? 1.0f / l : 0.f;
  for (int c = threadIdx.x; c < D; c += blockDim.x) {
    float o = 0.f;
    for (int s = 0; s < a.S; ++s) {
      const float ms = a.part_ml[(p0 + (size_t)s * a.M) * 2];
      if (ms != -INFINITY) o += a.part_acc[(p0 + (size_t)s * a.M) * D + c] * __expf(ms - mx);
    }
    a.out[(((size_t)b * a.M + r) * a.H + h) * D + c] = f2bf(o * inv);
  }
}

}  // namespace bita
