// Tree-based attention (Sec. 3.2, Fig. 6) on tensor cores, split over the key sequence.
//
// Keys of one (sequence, kv head): cache slots [0, C) are the context every row sees, slots
// [C, C+M) are the block's own rows (seen according to the ancestor bitmask, which the CTA keeps
// in shared memory), and the layer's P prompt-prefix keys (a separate buffer) are seen by mask
// rows only (Sec. 3.1).  They are walked in chunks of 64 keys; the chunks are dealt out evenly to
// `S` slices.  One CTA = one query head x one slice x up to 128 query rows; each warp owns 16 rows
// and keeps their running maximum, running sum and output accumulator in registers (online
// softmax, quad shuffles for the row reductions), K/V chunks are double-buffered in shared memory
// with cp.async, Q.K^T and P.V run as bf16 m16n8k16 MMAs with fp32 accumulation.  A single slice
// writes the output itself.  Several slices leave partial results (running maximum, running sum,
// unnormalised output) that are merged in slice order: inside the kernel when all CTAs of the
// launch are resident together (`sync` given: each slice merges an equal share of its row tile's
// rows once all slices of the tile have arrived), else by k_attn_merge.
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
  int32_t warps;             // warps per CTA = min(8, ceil(M / 16))
  int32_t row_tiles;         // ceil(M / (16 * warps))
  float scale_log2;          // log2(e) / sqrt(D)
  int32_t* sync;             // in-kernel merge: [2][B*H*row_tiles] arrival / departure counters, zero
                             // before the launch and left zero; null = partial results only
  int32_t* status;           // sticky error word for a wait that ran out (may be null)
};

constexpr unsigned long long ATT_WAIT_LIMIT_NS = 2000000000ull;

// Merged, normalised output of one row from its S partial results (slice order).  `lane` owns
// D / 32 consecutive features.
template <int D>
__device__ __forceinline__ void attn_merge_row(const AttnArgs& a, int b, int h, int gr, int lane) {
  constexpr int VW = D / 32;
  const size_t p0 = (((size_t)b * a.H + h) * a.S) * a.M + gr;
  float ms[8], ls[8], v[8][VW];
#pragma unroll
  for (int s = 0; s < 8; ++s) {
    if (s < a.S) {
      const size_t pi = p0 + (size_t)s * a.M;
      const float2 ml = __ldcg(reinterpret_cast<const float2*>(a.part_ml + pi * 2));
      ms[s] = ml.x;
      ls[s] = ml.y;
      if (VW == 4) {
        const float4 t = __ldcg(reinterpret_cast<const float4*>(a.part_acc + pi * D) + lane);
        v[s][0] = t.x; v[s][1] = t.y; v[s][VW - 2] = t.z; v[s][VW - 1] = t.w;
      } else {
        const float2 t = __ldcg(reinterpret_cast<const float2*>(a.part_acc + pi * D) + lane);
        v[s][0] = t.x; v[s][1] = t.y;
      }
    } else {
      ms[s] = -INFINITY;
      ls[s] = 0.f;
#pragma unroll
      for (int e = 0; e < VW; ++e) v[s][e] = 0.f;
    }
  }
  float mx = -INFINITY;
#pragma unroll
  for (int s = 0; s < 8; ++s) mx = fmaxf(mx, ms[s]);
  float l = 0.f, o[VW];
#pragma unroll
  for (int e = 0; e < VW; ++e) o[e] = 0.f;
#pragma unroll
  for (int s = 0; s < 8; ++s) {
    if (ms[s] == -INFINITY) continue;
    const float w = exp2f(ms[s] - mx);
    l += ls[s] * w;
#pragma unroll
    for (int e = 0; e < VW; ++e) o[e] += v[s][e] * w;
  }
  const float inv = l > 0.f ? 1.0f / l : 0.f;
  bf16* dst = a.out + (((size_t)b * a.M + gr) * a.H + h) * D + lane * VW;
#pragma unroll
  for (int e = 0; e < VW; e += 2)
    *reinterpret_cast<__nv_bfloat162*>(dst + e) = __floats2bfloat162_rn(o[e] * inv, o[e + 1] * inv);
}

constexpr int ATT_KEYS = 64;   // keys per chunk

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;   // 0 source bytes = fill the 16 bytes with zeros
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// Byte offset of 16-byte chunk `c` of row `r` in a [rows][D] bf16 tile whose chunks are XOR-swizzled
// by the row index (conflict-free ldmatrix).
template <int D>
__device__ __forceinline__ uint32_t swz(int r, int c) {
  return (uint32_t)(r * (D * 2) + ((c ^ (r & 7)) << 4));
}

// MAXW = most warps a CTA of this instantiation is launched with: blocks of up to 5 warps (80 query
// rows, the 69-row step block) are compiled to fit two per SM.
template <int D, int MAXW>
__global__ void __launch_bounds__(MAXW * 32, MAXW <= 5 ? 2 : 1) k_attn_tc(AttnArgs a) {
  constexpr int CH = D / 8;                  // 16-byte chunks per row
  constexpr int NT_S = ATT_KEYS / 8;         // score n-tiles per chunk
  constexpr int NT_O = D / 8;                // output n-tiles
  constexpr int KS_Q = D / 16;               // k-steps of Q.K^T
  constexpr int KS_P = ATT_KEYS / 16;        // k-steps of P.V
  extern __shared__ __align__(128) uint8_t smem[];
  pdl_launch();
  const int h = blockIdx.x, s = blockIdx.y;
  const int b = blockIdx.z / a.row_tiles, rt = blockIdx.z - b * a.row_tiles;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int nthreads = blockDim.x;
  const int rows_cta = a.warps * 16;
  const int row0 = rt * rows_cta;
  const int kvh = h / (a.H / a.H_kv);
  const int C = a.ctx_len[b];
  const int n_cache = C + a.M;                                  // cache keys in play
  const int cache_chunks = (n_cache + ATT_KEYS - 1) / ATT_KEYS;
  const bool has_prompt = a.P > 0 && a.prompt_k && a.prompt_v && a.sees_prompt;
  const int n_chunks = cache_chunks + (has_prompt ? 1 : 0);
  const int c_begin = (int)((long)n_chunks * s / a.S), c_end = (int)((long)n_chunks * (s + 1) / a.S);

  uint8_t* q_s = smem;                                          // [rows_cta][D]
  uint8_t* kv_s = smem + (size_t)rows_cta * D * 2;              // 2 x (K chunk, V chunk)
  constexpr int TILE_BYTES = ATT_KEYS * D * 2;
  uint32_t* vis_s = reinterpret_cast<uint32_t*>(kv_s + 4 * TILE_BYTES);   // [rows_cta][W]
  uint8_t* sp_s = reinterpret_cast<uint8_t*>(vis_s + (size_t)rows_cta * a.W);

  const bf16* kb = a.k + ((size_t)b * a.H_kv + kvh) * (size_t)a.C_max * D;
  const bf16* vb = a.v + ((size_t)b * a.H_kv + kvh) * (size_t)a.C_max * D;
  const bf16* pk = has_prompt ? a.prompt_k + (size_t)kvh * a.P * D : nullptr;
  const bf16* pv = has_prompt ? a.prompt_v + (size_t)kvh * a.P * D : nullptr;

  // ---- stage visibility words and prompt flags (fixed by the tree template)
  for (int i = threadIdx.x; i < rows_cta * a.W; i += nthreads) {
    const int r = i / a.W, w = i - r * a.W;
    const int gr = row0 + r;
    vis_s[i] = gr < a.M ? a.vis[(size_t)b * a.vis_batch_stride + (size_t)gr * a.W + w] : 0u;
  }
  for (int i = threadIdx.x; i < rows_cta; i += nthreads) {
    const int gr = row0 + i;
    sp_s[i] = (has_prompt && gr < a.M) ? a.sees_prompt[(size_t)b * a.sp_batch_stride + gr] : 0;
  }

  auto load_chunk = [&](int ci, int buf) {
    uint8_t* ks = kv_s + (size_t)buf * 2 * TILE_BYTES;
    uint8_t* vs = ks + TILE_BYTES;
    const bool is_prompt = ci >= cache_chunks;
    const int key0 = is_prompt ? 0 : ci * ATT_KEYS;
    const int limit = is_prompt ? a.P : n_cache;
    const bf16* ksrc = is_prompt ? pk : kb;
    const bf16* vsrc = is_prompt ? pv : vb;
    for (int i = threadIdx.x; i < ATT_KEYS * CH; i += nthreads) {
      const int r = i / CH, c = i - r * CH;
      const bool valid = key0 + r < limit;
      const size_t off = (size_t)(valid ? key0 + r : 0) * D + c * 8;
      cp_async16(smem_u32(ks) + swz<D>(r, c), ksrc + off, valid);
      cp_async16(smem_u32(vs) + swz<D>(r, c), vsrc + off, valid);
    }
  };

  // What does not depend on the kernel before this one is requested before waiting for it: the
  // context slots [0, C) were written by earlier passes and the prompt prefix is a weight, so a
  // chunk without block rows can be on its way while the projection that writes q and the block's
  // own k, v is still finishing.  Up to two chunks (both buffers) are requested ahead.
  auto early = [&](int ci) { return ci >= cache_chunks || (ci + 1) * ATT_KEYS <= C; };
  int issued = c_begin;                                         // chunks below this index are requested
  while (issued < c_end && issued < c_begin + 2 && early(issued)) {
    load_chunk(issued, issued - c_begin);
    cp_async_commit();
    ++issued;
  }
  pdl_wait();
  // ---- stage the Q rows
  for (int i = threadIdx.x; i < rows_cta * CH; i += nthreads) {
    const int r = i / CH, c = i - r * CH;
    const int gr = row0 + r;
    const bool valid = gr < a.M;
    const bf16* src = a.q + (((size_t)b * a.M + (valid ? gr : 0)) * a.H + h) * D + c * 8;
    cp_async16(smem_u32(q_s) + swz<D>(r, c), src, valid);
  }
  if (issued == c_begin && c_begin < c_end) {
    load_chunk(c_begin, 0);
    ++issued;
  }
  cp_async_commit();

  float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
  float o[NT_O][4];
#pragma unroll
  for (int j = 0; j < NT_O; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
  uint32_t qf[KS_Q][4];
  const int lr_a = warp * 16 + g, lr_b = lr_a + 8;              // this thread's two rows within the CTA
  const float sc = a.scale_log2;

  for (int ci = c_begin; ci < c_end; ++ci) {
    const int buf = (ci - c_begin) & 1;
    if (ci + 1 < c_end && ci + 1 >= issued) load_chunk(ci + 1, buf ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (ci == c_begin) {
      // Q fragments (rows warp*16 .. +15), once
#pragma unroll
      for (int kk = 0; kk < KS_Q; ++kk) {
        const int r = warp * 16 + (lane & 15), c = kk * 2 + (lane >> 4);
        ldsm_x4(smem_u32(q_s) + swz<D>(r, c), qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3]);
      }
    }
    const uint32_t ks = smem_u32(kv_s + (size_t)buf * 2 * TILE_BYTES);
    const uint32_t vs = ks + TILE_BYTES;
    // ---- scores S = Q K^T for 64 keys
    float sacc[NT_S][4];
#pragma unroll
    for (int j = 0; j < NT_S; ++j) { sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < KS_Q; ++kk) {
#pragma unroll
      for (int j = 0; j < NT_S; j += 2) {
        uint32_t b0, b1, b2, b3;
        const int r = j * 8 + (lane & 7) + ((lane >> 4) << 3), c = kk * 2 + ((lane >> 3) & 1);
        ldsm_x4(ks + swz<D>(r, c), b0, b1, b2, b3);
        mma_bf16(sacc[j], qf[kk], b0, b1);
        mma_bf16(sacc[j + 1], qf[kk], b2, b3);
      }
    }
    // ---- visibility
    const bool is_prompt = ci >= cache_chunks;
    const int key0 = is_prompt ? 0 : ci * ATT_KEYS;
    if (is_prompt) {
      const bool va = sp_s[lr_a] != 0, vb_ = sp_s[lr_b] != 0;
#pragma unroll
      for (int j = 0; j < NT_S; ++j) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const bool in = j * 8 + 2 * t + e < a.P;
          if (!(in && va)) sacc[j][e] = -INFINITY;
          if (!(in && vb_)) sacc[j][2 + e] = -INFINITY;
        }
      }
    } else if (key0 + ATT_KEYS > C) {
      const uint32_t* wa = vis_s + (size_t)lr_a * a.W;
      const uint32_t* wb = vis_s + (size_t)lr_b * a.W;
#pragma unroll
      for (int j = 0; j < NT_S; ++j) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int key = key0 + j * 8 + 2 * t + e;
          bool oka = true, okb = true;
          if (key >= n_cache) oka = okb = false;
          else if (key >= C) {
            const int jj = key - C;
            oka = (wa[jj >> 5] >> (jj & 31)) & 1u;
            okb = (wb[jj >> 5] >> (jj & 31)) & 1u;
          }
          if (!oka) sacc[j][e] = -INFINITY;
          if (!okb) sacc[j][2 + e] = -INFINITY;
        }
      }
    }
    // ---- online softmax (rows g and g + 8 of this warp's 16)
    float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
    for (int j = 0; j < NT_S; ++j) {
      mx_a = fmaxf(mx_a, fmaxf(sacc[j][0], sacc[j][1]));
      mx_b = fmaxf(mx_b, fmaxf(sacc[j][2], sacc[j][3]));
    }
    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
    const float mn_a = fmaxf(m_a, mx_a * sc), mn_b = fmaxf(m_b, mx_b * sc);
    const float sub_a = mn_a == -INFINITY ? 0.f : mn_a, sub_b = mn_b == -INFINITY ? 0.f : mn_b;
    const float corr_a = exp2f(m_a - sub_a), corr_b = exp2f(m_b - sub_b);
    m_a = mn_a;
    m_b = mn_b;
    l_a *= corr_a;
    l_b *= corr_b;
#pragma unroll
    for (int j = 0; j < NT_O; ++j) { o[j][0] *= corr_a; o[j][1] *= corr_a; o[j][2] *= corr_b; o[j][3] *= corr_b; }
    uint32_t pf[KS_P][4];
#pragma unroll
    for (int j = 0; j < NT_S; ++j) {
      const float p0 = exp2f(sacc[j][0] * sc - sub_a), p1 = exp2f(sacc[j][1] * sc - sub_a);
      const float p2 = exp2f(sacc[j][2] * sc - sub_b), p3 = exp2f(sacc[j][3] * sc - sub_b);
      l_a += p0 + p1;
      l_b += p2 + p3;
      pf[j >> 1][(j & 1) * 2] = pack_bf16(p0, p1);
      pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    // ---- O += P V
#pragma unroll
    for (int kk = 0; kk < KS_P; ++kk) {
#pragma unroll
      for (int j = 0; j < NT_O; j += 2) {
        uint32_t b0, b1, b2, b3;
        const int r = kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), c = j + (lane >> 4);
        ldsm_x4_t(vs + swz<D>(r, c), b0, b1, b2, b3);
        mma_bf16(o[j], pf[kk], b0, b1);
        mma_bf16(o[j + 1], pf[kk], b2, b3);
      }
    }
    __syncthreads();                                            // the buffer is refilled two iterations later
  }
  cp_async_wait<0>();

  l_a += __shfl_xor_sync(0xffffffffu, l_a, 1);
  l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
  l_b += __shfl_xor_sync(0xffffffffu, l_b, 1);
  l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
  const int gr_a = row0 + lr_a, gr_b = row0 + lr_b;
  if (a.S == 1) {
    // ---- the only slice: normalise and write the output
    const float inv_a = l_a > 0.f ? 1.0f / l_a : 0.f, inv_b = l_b > 0.f ? 1.0f / l_b : 0.f;
    if (gr_a < a.M) {
      bf16* dst = a.out + (((size_t)b * a.M + gr_a) * a.H + h) * D;
#pragma unroll
      for (int j = 0; j < NT_O; ++j)
        *reinterpret_cast<__nv_bfloat162*>(dst + j * 8 + 2 * t) = __floats2bfloat162_rn(o[j][0] * inv_a, o[j][1] * inv_a);
    }
    if (gr_b < a.M) {
      bf16* dst = a.out + (((size_t)b * a.M + gr_b) * a.H + h) * D;
#pragma unroll
      for (int j = 0; j < NT_O; ++j)
        *reinterpret_cast<__nv_bfloat162*>(dst + j * 8 + 2 * t) = __floats2bfloat162_rn(o[j][2] * inv_b, o[j][3] * inv_b);
    }
    return;
  }
  // ---- partial results of this slice
  const size_t pbase = (((size_t)b * a.H + h) * a.S + s) * a.M;
  if (gr_a < a.M) {
    if (t == 0) { a.part_ml[(pbase + gr_a) * 2] = m_a; a.part_ml[(pbase + gr_a) * 2 + 1] = l_a; }
    float* dst = a.part_acc + (pbase + gr_a) * D;
#pragma unroll
    for (int j = 0; j < NT_O; ++j) *reinterpret_cast<float2*>(dst + j * 8 + 2 * t) = make_float2(o[j][0], o[j][1]);
  }
  if (gr_b < a.M) {
    if (t == 0) { a.part_ml[(pbase + gr_b) * 2] = m_b; a.part_ml[(pbase + gr_b) * 2 + 1] = l_b; }
    float* dst = a.part_acc + (pbase + gr_b) * D;
#pragma unroll
    for (int j = 0; j < NT_O; ++j) *reinterpret_cast<float2*>(dst + j * 8 + 2 * t) = make_float2(o[j][2], o[j][3]);
  }
  if (!a.sync) return;                                          // k_attn_merge follows

  // ---- merge inside the kernel: all slices of this (sequence, head, row tile) are resident CTAs,
  // none of which waits before its partial results are out, so the wait ends; bounded all the same.
  const int n_sync = a.B * a.H * a.row_tiles;
  int32_t* arrived = a.sync + ((size_t)b * a.H + h) * a.row_tiles + rt;
  int32_t* departed = arrived + n_sync;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    atomicAdd(arrived, 1);
    unsigned long long w0 = 0;
    bool ok = true;
    for (uint32_t spin = 0;; ++spin) {
      int seen;
      asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(arrived) : "memory");
      if (seen >= a.S) break;
      if ((spin & 63u) == 63u) {
        unsigned long long now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
        if (w0 == 0) w0 = now;
        else if (now - w0 > ATT_WAIT_LIMIT_NS) { ok = false; break; }
      }
    }
    if (!ok && a.status) atomicExch(a.status, BITA_ERR_TIMEOUT);
    __threadfence();
  }
  __syncthreads();
  const int rows_here = min(rows_cta, a.M - row0);              // valid rows of this row tile
  const int r_lo = (int)((long)rows_here * s / a.S), r_hi = (int)((long)rows_here * (s + 1) / a.S);
  for (int r = r_lo + warp; r < r_hi; r += a.warps) attn_merge_row<D>(a, b, h, row0 + r, lane);
  __syncthreads();
  if (threadIdx.x == 0) {
    const int old = atomicAdd(departed, 1);
    if (old == a.S - 1) { *arrived = 0; *departed = 0; }         // ready for the next launch
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
