// Tree-based attention (Sec. 3.2, Fig. 6) on the tcgen05 tensor cores.
//
// Same interface, key enumeration, slicing and partial-result format as attention_tc.cuh; what
// differs is the inner engine.  One CTA = one query head x one key slice x up to 128 query rows.
// Keys are walked in chunks of 128:
//   S = Q K^T      one UMMA chain, M = 128 (query rows), N = 128 (keys), K = D; Q and the K chunk
//                  sit in shared memory as K-major 128-byte-swizzled tiles; S lands in TMEM with
//                  lane = query row, column = key (two S buffers alternate);
//   softmax        thread r of the four softmax warps owns query row r: it reads its row of S
//                  from TMEM, applies the visibility rule (context / ancestor bitmask / prompt
//                  prefix), keeps the running maximum and sum (online softmax, log2 domain),
//                  writes P = exp2(..) as bf16 into a K-major shared-memory tile and, when the
//                  maximum moved, rescales its row of the output accumulator in TMEM;
//   O += P V       second UMMA chain, M = 128, N = D, K = 128 keys; the V chunk is used as it
//                  lies in the cache ([key][D], i.e. MN-major for this product): the same staging
//                  layout serves K (K-major for Q K^T) and V (MN-major for P V).
// Roles: warps 0-3 softmax (TMEM lane group = warp), warp 4 issues the MMAs (one lane), warp 5
// stages Q and the K/V chunks with cp.async (two chunk buffers).  Everything is handed over
// through mbarriers with bounded waits; a wait that runs out raises the status word, the kernel
// drains and frees its TMEM.
#pragma once

#include "attention_tc.cuh"
#include "gemm_tc.cuh"

namespace bita {

constexpr int AU_KEYS = 128;        // keys per chunk
constexpr int AU_ROWS = 128;        // query rows per CTA
constexpr int AU_THREADS = 192;
constexpr int AU_ATOM = AU_ROWS * 128;   // bytes of one 128-row x 64-element swizzle atom column

// MN-major operand (rows of the staged tile = K index, 64 elements of MN per 128-byte row):
// groups of 8 K rows are 1024 bytes apart, the next 64 MN elements `lbo_bytes` further.
__device__ __forceinline__ uint64_t umma_smem_desc_mn(uint32_t addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
      "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
      "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
      "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])),
      "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
      : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_cta(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Byte offset of element (row r, 16-byte chunk c) in a tile staged as 64-element-wide swizzle atoms.
__device__ __forceinline__ uint32_t au_off(int r, int c) {
  return (uint32_t)((c >> 3) * AU_ATOM + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

template <int D>
__global__ void __launch_bounds__(AU_THREADS, 1) k_attn_umma(AttnArgs a) {
  constexpr int CH = D / 8;                         // 16-byte chunks per row
  constexpr int TILE = (D / 64) * AU_ATOM;          // bytes of a staged [128][D] tile
  constexpr uint32_t COL_S = 0, COL_O = 2 * AU_KEYS;
  constexpr uint32_t TMEM_COLS = 512;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_kv_full[2], bar_kv_empty[2], bar_s_full[2], bar_s_free[2], bar_p_full, bar_pv_done;
  __shared__ uint32_t tmem_slot;
  __shared__ int32_t status_local;                  // stands in when the caller gave no status word

  const int h = blockIdx.x, s = blockIdx.y;
  const int b = blockIdx.z / a.row_tiles, rt = blockIdx.z - b * a.row_tiles;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = rt * AU_ROWS;
  const int kvh = h / (a.H / a.H_kv);

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_s = base, kv_s = base + TILE, p_s = base + TILE + 4 * TILE;   // kv: 2 x (K tile, V tile)

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bar_kv_full[i]), 1);
      mbar_init(smem_u32(&bar_kv_empty[i]), 1);
      mbar_init(smem_u32(&bar_s_full[i]), 1);
      mbar_init(smem_u32(&bar_s_free[i]), 128);
    }
    mbar_init(smem_u32(&bar_p_full), 128);
    mbar_init(smem_u32(&bar_pv_done), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  int32_t* status = a.status ? a.status : &status_local;
  if (threadIdx.x == 0) pdl_launch();

  // ---- key chunks of this slice (the context length was settled by an earlier pass)
  const int C = a.ctx_len[b];
  const int n_cache = C + a.M;
  const int cache_chunks = (n_cache + AU_KEYS - 1) / AU_KEYS;
  const bool has_prompt = a.P > 0 && a.prompt_k && a.prompt_v && a.sees_prompt;
  const int n_chunks = cache_chunks + (has_prompt ? 1 : 0);
  const int c_begin = (int)((long)n_chunks * s / a.S), c_end = (int)((long)n_chunks * (s + 1) / a.S);
  const int n = c_end - c_begin;

  if (warp == 5) {
    // ---------------- loader: Q once, then K/V chunks into the two chunk buffers
    const bf16* kb = a.k + ((size_t)b * a.H_kv + kvh) * (size_t)a.C_max * D;
    const bf16* vb = a.v + ((size_t)b * a.H_kv + kvh) * (size_t)a.C_max * D;
    const bf16* pk = has_prompt ? a.prompt_k + (size_t)kvh * a.P * D : nullptr;
    const bf16* pv = has_prompt ? a.prompt_v + (size_t)kvh * a.P * D : nullptr;
    auto load_chunk = [&](int i) {
      const int ci = c_begin + i;
      const uint32_t ks = kv_s + (uint32_t)(i & 1) * 2 * TILE, vs = ks + TILE;
      const bool is_prompt = ci >= cache_chunks;
      const int key0 = is_prompt ? 0 : ci * AU_KEYS;
      const int limit = is_prompt ? a.P : n_cache;
      const bf16* ksrc = is_prompt ? pk : kb;
      const bf16* vsrc = is_prompt ? pv : vb;
      for (int j = lane; j < AU_KEYS * CH; j += 32) {
        const int r = j / CH, c = j - r * CH;
        const bool valid = key0 + r < limit;
        const size_t off = (size_t)(valid ? key0 + r : 0) * D + c * 8;
        cp_async16(ks + au_off(r, c), ksrc + off, valid);
        cp_async16(vs + au_off(r, c), vsrc + off, valid);
      }
    };
    // chunks without block rows depend on nothing the previous kernel writes
    auto early = [&](int i) { const int ci = c_begin + i; return ci >= cache_chunks || (ci + 1) * AU_KEYS <= C; };
    int issued = 0;
    while (issued < n && issued < 2 && early(issued)) { load_chunk(issued); ++issued; }
    pdl_wait();
    for (int j = lane; j < AU_ROWS * CH; j += 32) {
      const int r = j / CH, c = j - r * CH;
      const int gr = row0 + r;
      const bool valid = gr < a.M;
      const bf16* src = a.q + (((size_t)b * a.M + (valid ? gr : 0)) * a.H + h) * D + c * 8;
      cp_async16(q_s + au_off(r, c), src, valid);
    }
    if (issued == 0 && n > 0) { load_chunk(0); issued = 1; }
    cp_async_commit();
    cp_async_wait<0>();
    fence_async_smem();
    __syncwarp();
    if (lane == 0) {
      for (int i = 0; i < issued; ++i) mbar_arrive_cta(smem_u32(&bar_kv_full[i]));
    }
    bool ok = true;
    for (int i = issued; i < n && ok; ++i) {
      // the buffer was last used by chunk i - 2: free once its P V product has completed
      ok = mbar_wait(smem_u32(&bar_kv_empty[i & 1]), ((uint32_t)(i >> 1) & 1u) ^ 1u, status);
      if (!ok) break;
      load_chunk(i);
      cp_async_commit();
      cp_async_wait<0>();
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive_cta(smem_u32(&bar_kv_full[i & 1]));
    }
  } else if (warp == 4) {
    // ---------------- MMA issuer
    if (lane == 0 && n > 0) {
      const uint32_t idesc_s = umma_idesc(AU_KEYS);                       // S: N = keys of a chunk
      const uint32_t idesc_o = umma_idesc(D) | (1u << 16);                // O: N = D, B operand MN-major
      bool ok = true;
      auto issue_s = [&](int i) {
        const uint32_t ks = kv_s + (uint32_t)(i & 1) * 2 * TILE;
        const uint32_t d_tmem = tmem + COL_S + (uint32_t)(i & 1) * AU_KEYS;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint64_t da = umma_smem_desc(q_s + (kk >> 2) * AU_ATOM) + (uint64_t)(2 * (kk & 3));
          const uint64_t db = umma_smem_desc(ks + (kk >> 2) * AU_ATOM) + (uint64_t)(2 * (kk & 3));
          umma_bf16(d_tmem, da, db, idesc_s, kk > 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&bar_s_full[i & 1]));
      };
      ok = mbar_wait(smem_u32(&bar_kv_full[0]), 0, status);
      tc_fence_after();
      if (ok) issue_s(0);
      for (int i = 0; i < n && ok; ++i) {
        if (i + 1 < n) {                                                  // S of the next chunk while this one is in softmax
          ok = mbar_wait(smem_u32(&bar_kv_full[(i + 1) & 1]), (uint32_t)((i + 1) >> 1) & 1u, status);
          if (ok && i + 1 >= 2)
            ok = mbar_wait(smem_u32(&bar_s_free[(i + 1) & 1]), ((uint32_t)((i + 1) >> 1) & 1u) ^ 1u, status);
          if (!ok) break;
          tc_fence_after();
          issue_s(i + 1);
        }
        ok = mbar_wait(smem_u32(&bar_p_full), (uint32_t)i & 1u, status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t vs = kv_s + (uint32_t)(i & 1) * 2 * TILE + TILE;
#pragma unroll
        for (int kk = 0; kk < AU_KEYS / 16; ++kk) {
          const uint64_t da = umma_smem_desc(p_s + (kk >> 2) * AU_ATOM) + (uint64_t)(2 * (kk & 3));
          const uint64_t db = umma_smem_desc_mn(vs + kk * 16 * 128, AU_ATOM);
          umma_bf16(tmem + COL_O, da, db, idesc_o, (i > 0 || kk > 0) ? 1u : 0u);
        }
        umma_commit(smem_u32(&bar_kv_empty[i & 1]));
        umma_commit(smem_u32(&bar_pv_done));
      }
    }
  } else {
    // ---------------- softmax: thread r owns query row r
    const int r = threadIdx.x;
    const int gr = row0 + r;
    const bool row_live = gr < a.M;
    const float sc = a.scale_log2;
    uint32_t visw[8];
#pragma unroll
    for (int w = 0; w < 8; ++w)
      visw[w] = (row_live && w < a.W) ? a.vis[(size_t)b * a.vis_batch_stride + (size_t)gr * a.W + w] : 0u;
    const bool sees_p = has_prompt && row_live && a.sees_prompt[(size_t)b * a.sp_batch_stride + gr] != 0;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int i = 0; i < n; ++i) {
      const int ci = c_begin + i;
      const bool is_prompt = ci >= cache_chunks;
      const int key0 = is_prompt ? 0 : ci * AU_KEYS;
      const bool all_vis = !is_prompt && key0 + AU_KEYS <= C && row_live;
      auto visible = [&](int j) -> bool {                       // key j of the chunk for this row
        if (is_prompt) return sees_p && j < a.P;
        const int key = key0 + j;
        if (key < C) return row_live;
        if (key >= n_cache) return false;
        const int jj = key - C;
        return (visw[jj >> 5] >> (jj & 31)) & 1u;
      };
      if (ok) ok = mbar_wait(smem_u32(&bar_s_full[i & 1]), (uint32_t)(i >> 1) & 1u, status);
      ok = __all_sync(0xffffffffu, ok);                         // warp-uniform from here on
      tc_fence_after();
      const uint32_t s_addr = lane_addr + COL_S + (uint32_t)(i & 1) * AU_KEYS;
      // pass 1: row maximum over the visible keys
      float mx = -INFINITY;
      for (int c0 = 0; c0 < AU_KEYS; c0 += 16) {
        float v[16];
        tmem_ld16(s_addr + (uint32_t)c0, v);
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (all_vis || visible(c0 + j)) mx = fmaxf(mx, v[j]);
      }
      const float m_new = fmaxf(m_run, mx * sc);
      const float sub = m_new == -INFINITY ? 0.f : m_new;
      const float corr = exp2f(m_run - sub);                    // 0 while nothing was seen before
      // P overwrites the tile the previous P V product reads, and the rescale touches its accumulator
      if (i > 0 && ok) ok = mbar_wait(smem_u32(&bar_pv_done), (uint32_t)(i - 1) & 1u, status);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      // pass 2: P = exp2(s * scale - max), row sum, bf16 tile
      float sum = 0.f;
      for (int c0 = 0; c0 < AU_KEYS; c0 += 16) {
        float v[16];
        tmem_ld16(s_addr + (uint32_t)c0, v);
        uint32_t pk[8];
#pragma unroll
        for (int j = 0; j < 16; j += 2) {
          const float p0 = (all_vis || visible(c0 + j)) ? exp2f(v[j] * sc - sub) : 0.f;
          const float p1 = (all_vis || visible(c0 + j + 1)) ? exp2f(v[j + 1] * sc - sub) : 0.f;
          sum += p0 + p1;
          pk[j >> 1] = pack_bf16x2(p0, p1);
        }
        const int cc = c0 >> 3;                                 // 16-byte chunk index of keys c0 .. c0+7
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(p_s + au_off(r, cc)), "r"(pk[0]), "r"(pk[1]),
                     "r"(pk[2]), "r"(pk[3])
                     : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(p_s + au_off(r, cc + 1)), "r"(pk[4]), "r"(pk[5]),
                     "r"(pk[6]), "r"(pk[7])
                     : "memory");
      }
      tc_fence_before();
      mbar_arrive_cta(smem_u32(&bar_s_free[i & 1]));            // this S buffer may be overwritten
      if (i > 0 && __any_sync(0xffffffffu, corr != 1.0f)) {
        // the maximum of some row of this warp moved: bring the accumulator rows to their new
        // reference (the TMEM instructions are warp-wide, so the whole warp takes the branch)
        for (int c0 = 0; c0 < D; c0 += 16) {
          float v[16];
          tmem_ld16(lane_addr + COL_O + (uint32_t)c0, v);
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] *= corr;
          tmem_st16(lane_addr + COL_O + (uint32_t)c0, v);
        }
        tmem_wait_st();
      }
      l_run = l_run * corr + sum;
      m_run = m_new;
      fence_async_smem();                                       // the P tile is read by the tensor core
      tc_fence_before();
      mbar_arrive_cta(smem_u32(&bar_p_full));
    }
    if (n > 0 && ok) ok = mbar_wait(smem_u32(&bar_pv_done), (uint32_t)(n - 1) & 1u, status);
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    pdl_wait();
    // ---- result of this slice: row r of O
    if (a.S == 1) {
      const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
      bf16* dst = a.out + (((size_t)b * a.M + (row_live ? gr : 0)) * a.H + h) * D;
      for (int c0 = 0; c0 < D; c0 += 16) {
        float v[16];
        if (n > 0 && ok) {
          tmem_ld16(lane_addr + COL_O + (uint32_t)c0, v);
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0.f;
        }
        if (row_live) {
          uint4 w0, w1;
          w0.x = pack_bf16x2(v[0] * inv, v[1] * inv);   w0.y = pack_bf16x2(v[2] * inv, v[3] * inv);
          w0.z = pack_bf16x2(v[4] * inv, v[5] * inv);   w0.w = pack_bf16x2(v[6] * inv, v[7] * inv);
          w1.x = pack_bf16x2(v[8] * inv, v[9] * inv);   w1.y = pack_bf16x2(v[10] * inv, v[11] * inv);
          w1.z = pack_bf16x2(v[12] * inv, v[13] * inv); w1.w = pack_bf16x2(v[14] * inv, v[15] * inv);
          *reinterpret_cast<uint4*>(dst + c0) = w0;
          *reinterpret_cast<uint4*>(dst + c0 + 8) = w1;
        }
      }
    } else {
      const size_t pbase = (((size_t)b * a.H + h) * a.S + s) * a.M;
      if (row_live) {
        a.part_ml[(pbase + gr) * 2] = m_run;
        a.part_ml[(pbase + gr) * 2 + 1] = l_run;
      }
      float* dst = a.part_acc + (pbase + (row_live ? gr : 0)) * D;
      for (int c0 = 0; c0 < D; c0 += 16) {
        float v[16];
        if (n > 0 && ok) {
          tmem_ld16(lane_addr + COL_O + (uint32_t)c0, v);
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0.f;
        }
        if (row_live) {
#pragma unroll
          for (int j = 0; j < 16; j += 4)
            *reinterpret_cast<float4*>(dst + c0 + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        }
      }
      __threadfence();
    }
  }

  // ---- merge inside the kernel (all slices resident), as in attention_tc.cuh
  tc_fence_before();
  __syncthreads();
  if (a.S > 1 && a.sync) {
    const int n_sync = a.B * a.H * a.row_tiles;
    int32_t* arrived = a.sync + ((size_t)b * a.H + h) * a.row_tiles + rt;
    int32_t* departed = arrived + n_sync;
    if (threadIdx.x == 0) {
      atomicAdd(arrived, 1);
      unsigned long long w0 = 0;
      bool ok = true;
      for (uint32_t spin = 0; ld_acquire_gpu(arrived) < a.S; ++spin) {
        if ((spin & 63u) == 63u) {
          const unsigned long long now = global_ns();
          if (w0 == 0) w0 = now;
          else if (now - w0 > TC_WAIT_LIMIT_NS) { ok = false; break; }
        }
      }
      if (!ok) atomicExch(status, BITA_ERR_TIMEOUT);
      __threadfence();
    }
    __syncthreads();
    const int rows_here = min(AU_ROWS, a.M - row0);
    const int r_lo = (int)((long)rows_here * s / a.S), r_hi = (int)((long)rows_here * (s + 1) / a.S);
    for (int r = r_lo + warp; r < r_hi; r += AU_THREADS / 32) attn_merge_row<D>(a, b, h, row0 + r, lane);
    __syncthreads();
    if (threadIdx.x == 0) {
      const int old = atomicAdd(departed, 1);
      if (old == a.S - 1) { *arrived = 0; *departed = 0; }
    }
  }
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace bita
