// Tree-based attention (Sec. 3.2, Fig. 6) on the tcgen05 tensor cores.
//
// One CTA = one query head x one key slice x RT row tiles of 128 query rows (RT = 2 for blocks of
// more than 128 rows, so that both tiles share every K/V chunk that is read; arguments, slicing
// and the partial-result format: attention_common.cuh).  Keys are walked in chunks of 128, the
// cache chunks first, the prompt-prefix chunk last; slice s takes chunks s, s + S, ...  Per chunk
// and row tile:
//   S = Q K^T      one UMMA chain, M = 128 (query rows), N = 128 (keys), K = D; Q and the K chunk
//                  sit in shared memory as K-major 128-byte-swizzled tiles; S lands in TMEM with
//                  lane = query row, column = key (two S buffers alternate);
//   softmax        two threads per query row (warps w and w + 4 reach the same TMEM lanes), each with
//                  64 of the chunk's 128 keys: it reads its half row of S from TMEM, applies the
//                  visibility rule (context / ancestor bitmask / prompt prefix), exchanges the
//                  half-row maximum with its partner through shared memory, keeps the running
//                  maximum and its half of the running sum (online softmax, log2 domain), writes
//                  P = exp2(..) as bf16 into a K-major shared-memory tile and, when the maximum
//                  moved, rescales its half of the row of the output accumulator in TMEM;
//   O += P V       second UMMA chain, M = 128, N = D, K = 128 keys; the V chunk is used as it
//                  lies in the cache ([key][D], i.e. MN-major for this product): the same staging
//                  layout serves K (K-major for Q K^T) and V (MN-major for P V).
// Roles: warps 0-7 softmax (TMEM lane group = warp % 4), warp 8 issues the MMAs (one lane), warp 9
// brings Q and the K/V chunks in with TMA (two chunk buffers; box = 64 features x 128 rows, 128-byte
// swizzle, no multicast) and clears the V rows past the last key before handing a chunk over.
// Everything is handed over through mbarriers with bounded waits; a wait that runs out raises the
// status word, the kernel drains and frees its TMEM.  Several key slices of one (sequence, head, row tile) run as one
// thread-block cluster and merge their partial results through distributed shared memory.
#pragma once

#include "attention_common.cuh"
#include "gemm_tc.cuh"

namespace bita {

constexpr int AU_KEYS = 128;        // keys per chunk
constexpr int AU_ROWS = 128;        // query rows per row tile
constexpr int AU_THREADS = 320;      // 8 softmax warps, MMA warp, loader warp
constexpr int AU_SOFTMAX = 256;      // softmax threads: two per query row
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

__device__ __forceinline__ void mbar_arrive_cta(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 3-D tiled TMA load global -> shared (no multicast), completion on an mbarrier.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}

// Tensor maps of one attention call.  q: (D, H, B*M) box (64, 1, 128); k, v: (D, C_max, B*H_kv) box
// (64, 128, 1); prompt_k, prompt_v: (D, P, H_kv) box (64, 128, 1) (copies of k, v when there is no prefix).
struct AttnMaps {
  CUtensorMap q, k, v, pk, pv;
};

// ---- cluster helpers: a peer CTA's shared memory and mbarriers
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t cta_rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(cta_rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t remote_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
// Bounded wait with cluster-scope acquire (the data were written by other CTAs of the cluster).
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, int32_t* status,
                                                  unsigned long long limit_ns) {
  unsigned long long t0 = 0;
  for (uint32_t i = 0;; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if ((i & 63u) == 63u) {
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) break;
    }
  }
  atomicExch(status, BITA_ERR_TIMEOUT);
  return false;
}
__device__ __forceinline__ float4 ld_dsmem_f4(uint32_t remote_addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote_addr));
  return v;
}
__device__ __forceinline__ float2 ld_dsmem_f2(uint32_t remote_addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(remote_addr));
  return v;
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Byte offset of element (row r, 16-byte chunk c) in a tile staged as 64-element-wide swizzle atoms.
__device__ __forceinline__ uint32_t au_off(int r, int c) {
  return (uint32_t)((c >> 3) * AU_ATOM + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

template <int D, int RT>
__global__ void __launch_bounds__(AU_THREADS, 1) k_attn_umma(const __grid_constant__ AttnMaps maps, AttnArgs a) {
  constexpr int CH = D / 8;                         // 16-byte chunks per row
  constexpr int TILE = (D / 64) * AU_ATOM;          // bytes of a staged [128][D] tile
  constexpr uint32_t COL_S = 0, COL_O = 2 * AU_KEYS;   // two S buffers, then RT output accumulators of D columns
  static_assert(2 * AU_KEYS + RT * D <= 512, "tensor memory");
  constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t PSTRIDE = (D + 4) * 4;         // bytes of a partial row in shared memory: m, l, pad, O[D]
  extern __shared__ uint8_t smem_raw[];
  // K and V tiles of a chunk buffer are handed over separately: a K tile is free again once its
  // Q K^T chain is done (long before the chunk's P V product), so the next K is on its way early.
  __shared__ __align__(8) uint64_t bar_k_full[2], bar_k_empty[2], bar_v_full[2], bar_v_empty[2];
  __shared__ __align__(8) uint64_t bar_s_full[2], bar_s_free[2], bar_p_full, bar_pv_done, bar_q, bar_vfix;
  __shared__ __align__(8) uint64_t bar_cl_in, bar_cl_out;      // cluster merge: partials in / reads done
  __shared__ uint32_t tmem_slot;
  __shared__ int32_t status_local;                  // stands in when the caller gave no status word
  __shared__ float xchg[2][AU_ROWS];                // [half][row]: half-row maxima (and, at the end, sums)

  const int h = blockIdx.x, s = blockIdx.y;
  const int b = blockIdx.z / a.row_tiles, rt = blockIdx.z - b * a.row_tiles;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = rt * RT * AU_ROWS;
  const int kvh = h / (a.H / a.H_kv);

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  // Q (RT tiles), 2 x (K tile, V tile), P
  const uint32_t q_s = base, kv_s = base + RT * TILE, p_s = kv_s + 4 * TILE;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bar_k_full[i]), 1);
      mbar_init(smem_u32(&bar_k_empty[i]), 1);
      mbar_init(smem_u32(&bar_v_full[i]), 1);
      mbar_init(smem_u32(&bar_v_empty[i]), 1);
      mbar_init(smem_u32(&bar_s_full[i]), 1);
      mbar_init(smem_u32(&bar_s_free[i]), AU_SOFTMAX);
    }
    mbar_init(smem_u32(&bar_q), 1);
    mbar_init(smem_u32(&bar_vfix), 1);
    mbar_init(smem_u32(&bar_cl_in), (uint32_t)a.S);
    mbar_init(smem_u32(&bar_cl_out), (uint32_t)a.S);
    mbar_init(smem_u32(&bar_p_full), AU_SOFTMAX);
    mbar_init(smem_u32(&bar_pv_done), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (a.S > 1 && a.cluster) {
    // peers arrive on this CTA's merge barriers: they must be initialised cluster-wide first
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  }
  const uint32_t tmem = tmem_slot;
  int32_t* status = a.status ? a.status : &status_local;
  const unsigned long long wait_ns = a.wait_ns;
  if (threadIdx.x == 0) pdl_launch();

  // ---- key chunks of this slice (the context length was settled by an earlier pass)
  const int C = a.ctx_len[(size_t)b * a.ctx_len_stride];
  const int n_cache = C + a.M;
  const int cache_chunks = (n_cache + AU_KEYS - 1) / AU_KEYS;
  const bool has_prompt = a.P > 0 && a.prompt_k && a.prompt_v && a.sees_prompt;
  const int n_chunks = cache_chunks + (has_prompt ? 1 : 0);
  // Chunks are dealt round-robin: slice s takes chunks s, s + S, s + 2S, ...  The chunks that hold
  // the block's own keys (the last cache chunks: not available before the dependency wait) thus go
  // to different slices, each of which has earlier chunks to work on first.
  const int n = s < n_chunks ? (n_chunks - s + a.S - 1) / a.S : 0;
  auto chunk_of = [&](int i) { return s + i * a.S; };
  // The tensor core and the softmax warps work in steps j = chunk * RT + row tile; S buffer j & 1.
  const int n_steps = n * RT;
  // The cache chunk that holds the last key may end in slots that were never written: their V rows
  // are cleared before the P V product (`fix` = index of that chunk within this slice, or -1).
  const int fix = (n_cache % AU_KEYS != 0 && cache_chunks - 1 >= s && (cache_chunks - 1 - s) % a.S == 0)
                      ? (cache_chunks - 1 - s) / a.S : -1;

  if (warp == 9) {
    // ---------------- loader (one lane issues; the warp clears the rows of the `fix` chunk)
    auto issue_tile = [&](int i, bool v_tile) {                  // lane 0 only
      const int ci = chunk_of(i);
      const uint32_t dst = kv_s + (uint32_t)(i & 1) * 2 * TILE + (v_tile ? TILE : 0);
      const bool is_prompt = ci >= cache_chunks;
      const uint32_t bar = smem_u32(v_tile ? &bar_v_full[i & 1] : &bar_k_full[i & 1]);
      const CUtensorMap* map = is_prompt ? (v_tile ? &maps.pv : &maps.pk) : (v_tile ? &maps.v : &maps.k);
      mbar_expect_tx(bar, (uint32_t)TILE);
#pragma unroll
      for (int hf = 0; hf < D / 64; ++hf)
        tma_load_3d(dst + hf * AU_ATOM, map, hf * 64, is_prompt ? 0 : ci * AU_KEYS, is_prompt ? kvh : b * a.H_kv + kvh, bar);
    };
    // chunks without block rows depend on nothing the previous kernel writes
    auto early = [&](int i) { const int ci = chunk_of(i); return ci >= cache_chunks || (ci + 1) * AU_KEYS <= C; };
    int k_issued = 0, v_issued = 0;
    while (k_issued < n && k_issued < 2 && early(k_issued)) {
      if (lane == 0) { issue_tile(k_issued, false); issue_tile(k_issued, true); }
      ++k_issued;
    }
    v_issued = k_issued;
    pdl_wait();
    if (lane == 0 && n > 0) {
      mbar_expect_tx(smem_u32(&bar_q), (uint32_t)(RT * TILE));
#pragma unroll
      for (int t = 0; t < RT; ++t) {
#pragma unroll
        for (int hf = 0; hf < D / 64; ++hf)
          tma_load_3d(q_s + t * TILE + hf * AU_ATOM, &maps.q, hf * 64, h, b * a.M + row0 + t * AU_ROWS, smem_u32(&bar_q));
      }
    }
    bool ok = true;
    if (k_issued == 0 && n > 0) {
      if (lane == 0) issue_tile(0, false);
      k_issued = 1;
    }
    // The MMA thread runs (per chunk, all row tiles) S(0), S(1), PV(0), S(2), PV(1), ...: K(j+1)
    // waits for the S of chunk j-1, then V(j) for the PV of chunk j-2, in that order.
    for (int j = 0; j < n && ok; ++j) {
      if (j + 1 < n && j + 1 >= k_issued) {
        if (j + 1 >= 2) ok = mbar_wait(smem_u32(&bar_k_empty[(j + 1) & 1]), ((uint32_t)((j + 1) >> 1) & 1u) ^ 1u, status, wait_ns);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (lane == 0) issue_tile(j + 1, false);
        k_issued = j + 2;
      }
      if (j >= v_issued) {
        if (j >= 2) ok = mbar_wait(smem_u32(&bar_v_empty[j & 1]), ((uint32_t)(j >> 1) & 1u) ^ 1u, status, wait_ns);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (lane == 0) issue_tile(j, true);
        v_issued = j + 1;
      }
      if (j == fix) {
        ok = mbar_wait(smem_u32(&bar_v_full[j & 1]), (uint32_t)(j >> 1) & 1u, status, wait_ns);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const int live_rows = n_cache - chunk_of(j) * AU_KEYS;
        const uint32_t vs = kv_s + (uint32_t)(j & 1) * 2 * TILE + TILE;
        for (int t = lane; t < (AU_KEYS - live_rows) * CH; t += 32) {
          const int r = live_rows + t / CH, c = t % CH;
          asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vs + au_off(r, c)), "r"(0u) : "memory");
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive_cta(smem_u32(&bar_vfix));
      }
    }
    if (!ok) {
      for (int i = 0; i < 64; ++i) __nanosleep(1000);            // let the copies in flight land
    }
  } else if (warp == 8) {
    // ---------------- MMA issuer
    if (lane == 0 && n > 0) {
      const uint32_t idesc_s = umma_idesc(AU_KEYS);                       // S: N = keys of a chunk
      const uint32_t idesc_o = umma_idesc(D) | (1u << 16);                // O: N = D, B operand MN-major
      bool ok = true;
      auto issue_s = [&](int j) {                                         // step j: chunk j / RT, row tile j % RT
        const int i = j / RT, t = j - i * RT;
        const uint32_t ks = kv_s + (uint32_t)(i & 1) * 2 * TILE;
        const uint32_t d_tmem = tmem + COL_S + (uint32_t)(j & 1) * AU_KEYS;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint64_t da = umma_smem_desc(q_s + t * TILE + (kk >> 2) * AU_ATOM) + (uint64_t)(2 * (kk & 3));
          const uint64_t db = umma_smem_desc(ks + (kk >> 2) * AU_ATOM) + (uint64_t)(2 * (kk & 3));
          umma_bf16(d_tmem, da, db, idesc_s, kk > 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&bar_s_full[j & 1]));
        if (t == RT - 1) umma_commit(smem_u32(&bar_k_empty[i & 1]));      // the K tile has served every row tile
      };
      ok = mbar_wait(smem_u32(&bar_q), 0, status, wait_ns);
      if (ok) ok = mbar_wait(smem_u32(&bar_k_full[0]), 0, status, wait_ns);
      tc_fence_after();
      if (ok) issue_s(0);
      for (int j = 0; j < n_steps && ok; ++j) {
        if (j + 1 < n_steps) {                                            // S of the next step while this one is in softmax
          const int i1 = (j + 1) / RT;
          if ((j + 1) % RT == 0) ok = mbar_wait(smem_u32(&bar_k_full[i1 & 1]), (uint32_t)(i1 >> 1) & 1u, status, wait_ns);
          if (ok && j + 1 >= 2)
            ok = mbar_wait(smem_u32(&bar_s_free[(j + 1) & 1]), ((uint32_t)((j + 1) >> 1) & 1u) ^ 1u, status, wait_ns);
          if (!ok) break;
          tc_fence_after();
          issue_s(j + 1);
        }
        const int i = j / RT, t = j - i * RT;
        ok = mbar_wait(smem_u32(&bar_p_full), (uint32_t)j & 1u, status, wait_ns);
        if (ok && t == 0) ok = mbar_wait(smem_u32(&bar_v_full[i & 1]), (uint32_t)(i >> 1) & 1u, status, wait_ns);
        if (ok && t == 0 && i == fix) ok = mbar_wait(smem_u32(&bar_vfix), 0, status, wait_ns);
        if (!ok) break;
        tc_fence_after();
        const uint32_t vs = kv_s + (uint32_t)(i & 1) * 2 * TILE + TILE;
#pragma unroll
        for (int kk = 0; kk < AU_KEYS / 16; ++kk) {
          const uint64_t da = umma_smem_desc(p_s + (kk >> 2) * AU_ATOM) + (uint64_t)(2 * (kk & 3));
          const uint64_t db = umma_smem_desc_mn(vs + kk * 16 * 128, AU_ATOM);
          umma_bf16(tmem + COL_O + (uint32_t)(t * D), da, db, idesc_o, (i > 0 || kk > 0) ? 1u : 0u);
        }
        if (t == RT - 1) umma_commit(smem_u32(&bar_v_empty[i & 1]));
        umma_commit(smem_u32(&bar_pv_done));
      }
    }
  } else {
    // ---------------- softmax: threads r and r + 128 share query row r of every row tile of the
    // CTA; thread half g takes keys [64 g, 64 g + 64) of a chunk and columns [g D/2, (g+1) D/2) of O
    const int r = threadIdx.x & (AU_ROWS - 1), g = threadIdx.x >> 7;
    constexpr int HK = AU_KEYS / 2, HD = D / 2;
    const float sc = a.scale_log2;
    int gr[RT];
    bool row_live[RT], sees_p[RT];
    constexpr int VW_MAX = BITA_MAX_ROWS / 32;                      // words of a row's ancestor bitmask
    uint32_t visw[RT][VW_MAX];
    float m_run[RT], l_run[RT];
#pragma unroll
    for (int t = 0; t < RT; ++t) {
      gr[t] = row0 + t * AU_ROWS + r;
      row_live[t] = gr[t] < a.M;
#pragma unroll
      for (int w = 0; w < VW_MAX; ++w) {
        visw[t][w] = (row_live[t] && w < a.W) ? a.vis[(size_t)b * a.vis_batch_stride + (size_t)gr[t] * a.W + w] : 0u;
        const int nb = a.M - 32 * w;                            // block rows this word can name
        if (nb < 32) visw[t][w] &= nb <= 0 ? 0u : ((1u << nb) - 1u);
      }
      sees_p[t] = has_prompt && row_live[t] && a.sees_prompt[(size_t)b * a.sp_batch_stride + gr[t]] != 0;
      m_run[t] = -INFINITY;
      l_run[t] = 0.f;                                           // this thread's half of the row sum
    }
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    bool ok = true;
    for (int j = 0; j < n_steps; ++j) {
      const int i = j / RT;
      const int ci = chunk_of(i);
      const bool is_prompt = ci >= cache_chunks;
      const int key0 = is_prompt ? 0 : ci * AU_KEYS;
      // this step's row tile (compile-time selects keep the per-tile state in registers)
      const bool second = RT > 1 && (j & 1);
      const bool live = second ? row_live[RT - 1] : row_live[0];
      const bool sp = second ? sees_p[RT - 1] : sees_p[0];
      const float m_old = second ? m_run[RT - 1] : m_run[0];
      const uint32_t o_addr = lane_addr + COL_O + (second ? (uint32_t)((RT - 1) * D) : 0u) + (uint32_t)(g * HD);
      const bool all_vis = !is_prompt && key0 + AU_KEYS <= C && live;
      // Visibility of this thread's 64 keys as two 32-bit words: context keys are seen by every
      // live row, block keys according to the row's ancestor bitmask (shifted to the key's place),
      // prompt keys by mask rows only; keys past the last one by nobody.
      uint32_t vm[2] = {0u, 0u};
      if (live && !all_vis) {
#pragma unroll
        for (int w2 = 0; w2 < 2; ++w2) {
          const int w = 2 * g + w2;                             // word of the chunk
          if (is_prompt) {
            const int nb = a.P - 32 * w;                        // prompt keys in this word
            vm[w2] = !sp || nb <= 0 ? 0u : (nb >= 32 ? 0xffffffffu : ((1u << nb) - 1u));
          } else {
            const int j0 = key0 + 32 * w - C;                   // block row index of the word's first key
            uint32_t word;
            if (j0 <= -32) {
              word = 0xffffffffu;                               // all context
            } else {
              // bits [j0, j0 + 32) of the row's bitmask (bits below 0 are context: ones)
              const int q = j0 >= 0 ? j0 >> 5 : -1, sh = j0 & 31;
              uint32_t lo = q < 0 ? 0xffffffffu : 0u, hi = 0u;
#pragma unroll
              for (int u = 0; u < VW_MAX; ++u) {
                const uint32_t vw = second ? visw[RT - 1][u] : visw[0][u];
                if (u == q) lo = vw;
                if (u == q + 1) hi = vw;
              }
              word = sh == 0 ? lo : __funnelshift_r(lo, hi, sh);
            }
            vm[w2] = word;
          }
        }
      }
      if (ok) ok = mbar_wait(smem_u32(&bar_s_full[j & 1]), (uint32_t)(j >> 1) & 1u, status, wait_ns);
      ok = __all_sync(0xffffffffu, ok);                         // warp-uniform from here on
      tc_fence_after();
      const uint32_t s_addr = lane_addr + COL_S + (uint32_t)(j & 1) * AU_KEYS + (uint32_t)(g * HK);
      // this thread's half row of scores into registers (one TMEM round trip); the buffer is free again
      float sv[HK];
      tmem_ld64(s_addr, sv);
      tc_fence_before();
      mbar_arrive_cta(smem_u32(&bar_s_free[j & 1]));
      float mx = -INFINITY;
      if (all_vis) {
#pragma unroll
        for (int e = 0; e < HK; ++e) mx = fmaxf(mx, sv[e]);
      } else {
#pragma unroll
        for (int e = 0; e < HK; ++e) {
          if (!((vm[e >> 5] >> (e & 31)) & 1u)) sv[e] = -INFINITY;   // exp2(-inf) = 0 below
          mx = fmaxf(mx, sv[e]);
        }
      }
      // the row maximum is the larger of the two halves': exchange through shared memory
      xchg[g][r] = mx;
      asm volatile("bar.sync 1, %0;" ::"n"(AU_SOFTMAX) : "memory");
      mx = fmaxf(mx, xchg[g ^ 1][r]);
      asm volatile("bar.sync 1, %0;" ::"n"(AU_SOFTMAX) : "memory");   // both have read: the slots may be rewritten
      const float m_new = fmaxf(m_old, mx * sc);
      const float sub = m_new == -INFINITY ? 0.f : m_new;
      const float corr = exp2f(m_old - sub);                    // 0 while nothing was seen before
      // P overwrites the tile the previous P V product reads, and the rescale touches an accumulator
      if (j > 0 && ok) ok = mbar_wait(smem_u32(&bar_pv_done), (uint32_t)(j - 1) & 1u, status, wait_ns);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      // P = exp2(s * scale - max), half-row sum, bf16 tile (this thread's 64 keys are one swizzle atom)
      float sum = 0.f;
#pragma unroll
      for (int c0 = 0; c0 < HK; c0 += 8) {
        uint32_t pk[4];
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
          const float p0 = ex2_approx(sv[c0 + e] * sc - sub), p1 = ex2_approx(sv[c0 + e + 1] * sc - sub);
          sum += p0 + p1;
          pk[e >> 1] = pack_bf16x2(p0, p1);
        }
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(p_s + au_off(r, g * 8 + (c0 >> 3))), "r"(pk[0]),
                     "r"(pk[1]), "r"(pk[2]), "r"(pk[3])
                     : "memory");
      }
      if (i > 0 && __any_sync(0xffffffffu, corr != 1.0f)) {
        // the maximum of some row of this warp moved: bring the accumulator rows to their new
        // reference (the TMEM instructions are warp-wide, so the whole warp takes the branch)
        float ov[HD];
        if constexpr (HD == 64) tmem_ld64(o_addr, ov); else tmem_ld32(o_addr, ov);
#pragma unroll
        for (int e = 0; e < HD; ++e) ov[e] *= corr;
        if constexpr (HD == 64) tmem_st64(o_addr, ov); else tmem_st32(o_addr, ov);
      }
      if (second) { l_run[RT - 1] = l_run[RT - 1] * corr + sum; m_run[RT - 1] = m_new; }
      else { l_run[0] = l_run[0] * corr + sum; m_run[0] = m_new; }
      fence_async_smem();                                       // the P tile is read by the tensor core
      tc_fence_before();
      mbar_arrive_cta(smem_u32(&bar_p_full));
    }
    if (n_steps > 0 && ok) ok = mbar_wait(smem_u32(&bar_pv_done), (uint32_t)(n_steps - 1) & 1u, status, wait_ns);
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    pdl_wait();
    // ---- result of this slice: this thread's half of row r of O, per row tile
#pragma unroll
    for (int t = 0; t < RT; ++t) {
      // the row sum is the sum of the two halves' (same reference maximum in both)
      xchg[g][r] = l_run[t];
      asm volatile("bar.sync 1, %0;" ::"n"(AU_SOFTMAX) : "memory");
      const float l_row = l_run[t] + xchg[g ^ 1][r];
      asm volatile("bar.sync 1, %0;" ::"n"(AU_SOFTMAX) : "memory");
      float ov[HD];
      const uint32_t o_addr = lane_addr + COL_O + (uint32_t)(t * D + g * HD);
      if (n_steps > 0 && ok) {
        if constexpr (HD == 64) tmem_ld64(o_addr, ov); else tmem_ld32(o_addr, ov);
      } else {
#pragma unroll
        for (int e = 0; e < HD; ++e) ov[e] = 0.f;
      }
      if (a.S == 1) {
        const float inv = l_row > 0.f ? 1.0f / l_row : 0.f;
        if (row_live[t]) {
          bf16* dst = a.out + (((size_t)b * a.M + gr[t]) * a.H + h) * D + g * HD;
#pragma unroll
          for (int c0 = 0; c0 < HD; c0 += 8) {
            uint4 w;
            w.x = pack_bf16x2(ov[c0] * inv, ov[c0 + 1] * inv);     w.y = pack_bf16x2(ov[c0 + 2] * inv, ov[c0 + 3] * inv);
            w.z = pack_bf16x2(ov[c0 + 4] * inv, ov[c0 + 5] * inv); w.w = pack_bf16x2(ov[c0 + 6] * inv, ov[c0 + 7] * inv);
            *reinterpret_cast<uint4*>(dst + c0) = w;
          }
        }
      } else if (a.cluster) {
        // partial result of this row into this CTA's shared memory (the chunk buffers and the P tile
        // are free: every copy into them has landed and every MMA that read them is complete)
        if (row_live[t]) {
          const uint32_t prow = kv_s + (uint32_t)(t * AU_ROWS + r) * PSTRIDE;
          if (g == 0) asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(prow), "f"(m_run[t]), "f"(l_row) : "memory");
#pragma unroll
          for (int e = 0; e < HD; e += 4)
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(prow + 16 + (g * HD + e) * 4), "f"(ov[e]),
                         "f"(ov[e + 1]), "f"(ov[e + 2]), "f"(ov[e + 3])
                         : "memory");
        }
      } else {
        const size_t pbase = (((size_t)b * a.H + h) * a.S + s) * a.M;
        if (row_live[t]) {
          if (g == 0) {
            a.part_ml[(pbase + gr[t]) * 2] = m_run[t];
            a.part_ml[(pbase + gr[t]) * 2 + 1] = l_row;
          }
          float* dst = a.part_acc + (pbase + gr[t]) * D + g * HD;
#pragma unroll
          for (int e = 0; e < HD; e += 4)
            *reinterpret_cast<float4*>(dst + e) = make_float4(ov[e], ov[e + 1], ov[e + 2], ov[e + 3]);
        }
      }
    }
    if (a.S > 1 && !a.cluster) __threadfence();
  }

  // ---- merge inside the cluster: the S slices of this (sequence, head, row tile) are the CTAs of
  // one cluster (rank = slice).  Each leaves its partial rows in its own shared memory, tells every
  // peer, and once all S are in merges an equal share of the rows, reading the peers' partials
  // through distributed shared memory, in slice order.  A second round of arrivals keeps every CTA
  // alive until its peers have finished reading it.  Both waits are bounded mbarrier waits.
  tc_fence_before();
  __syncthreads();
  if (a.S > 1 && a.cluster) {
    if (threadIdx.x == 0) {
      asm volatile("fence.acq_rel.cluster;" ::: "memory");
      for (int p = 0; p < a.S; ++p) mbar_arrive_remote(mapa_u32(smem_u32(&bar_cl_in), (uint32_t)p));
    }
    mbar_wait_cluster(smem_u32(&bar_cl_in), 0, status, wait_ns);
    constexpr int VW = D / 32;
    const int rows_here = min(RT * AU_ROWS, a.M - row0);
    const int r_lo = (int)((long)rows_here * s / a.S), r_hi = (int)((long)rows_here * (s + 1) / a.S);
    constexpr int NW = AU_THREADS / 32, RR = 3;                 // rows per warp whose loads fly together
    for (int r0 = r_lo + warp; r0 < r_hi; r0 += NW * RR) {
      float ms[RR][8], ls[RR][8], v[RR][8][VW];
#pragma unroll
      for (int u = 0; u < RR; ++u) {
        const int r = min(r0 + u * NW, r_hi - 1);               // clamped: surplus slots redo the last row
#pragma unroll
        for (int p = 0; p < 8; ++p) {
          ms[u][p] = -INFINITY;
          ls[u][p] = 0.f;
#pragma unroll
          for (int e = 0; e < VW; ++e) v[u][p][e] = 0.f;
          if (p < a.S) {
            const uint32_t prow = mapa_u32(kv_s + (uint32_t)r * PSTRIDE, (uint32_t)p);
            const float2 ml = ld_dsmem_f2(prow);
            ms[u][p] = ml.x;
            ls[u][p] = ml.y;
            if constexpr (VW == 4) {
              const float4 t = ld_dsmem_f4(prow + 16 + lane * 16);
              v[u][p][0] = t.x; v[u][p][1] = t.y; v[u][p][2] = t.z; v[u][p][3] = t.w;
            } else {
              const float2 t = ld_dsmem_f2(prow + 16 + lane * 8);
              v[u][p][0] = t.x; v[u][p][1] = t.y;
            }
          }
        }
      }
#pragma unroll
      for (int u = 0; u < RR; ++u) {
        const int r = r0 + u * NW;
        if (r >= r_hi) break;
        float mx = -INFINITY;
#pragma unroll
        for (int p = 0; p < 8; ++p) mx = fmaxf(mx, ms[u][p]);
        float l = 0.f, o[VW];
#pragma unroll
        for (int e = 0; e < VW; ++e) o[e] = 0.f;
#pragma unroll
        for (int p = 0; p < 8; ++p) {
          if (ms[u][p] == -INFINITY) continue;
          const float w = exp2f(ms[u][p] - mx);
          l += ls[u][p] * w;
#pragma unroll
          for (int e = 0; e < VW; ++e) o[e] += v[u][p][e] * w;
        }
        const float inv = l > 0.f ? 1.0f / l : 0.f;
        bf16* dst = a.out + (((size_t)b * a.M + row0 + r) * a.H + h) * D + lane * VW;
#pragma unroll
        for (int e = 0; e < VW; e += 2)
          *reinterpret_cast<__nv_bfloat162*>(dst + e) = __floats2bfloat162_rn(o[e] * inv, o[e + 1] * inv);
      }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int p = 0; p < a.S; ++p) mbar_arrive_remote(mapa_u32(smem_u32(&bar_cl_out), (uint32_t)p));
    }
    mbar_wait_cluster(smem_u32(&bar_cl_out), 0, status, wait_ns);
  }
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace bita
