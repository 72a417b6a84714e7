// Several projections of one layer as ONE persistent kernel.
//
// The per-projection kernel (gemm_tc.cuh) streams at HBM rate inside its main loop but pays a few
// microseconds of start-up and tail per launch; at small model widths those fixed costs are as
// large as the streaming time.  Here up to four projections that depend on one another (O ->
// gate/up -> down -> next layer's q/k/v) run as phases of one grid of resident CTAs:
//   * the TMA producer walks the CTA's whole sequence of weight tiles, phase after phase, and is
//     only held back by the ring; the weight tiles of the next phase are on their way while the
//     current phase finishes (weights depend on nothing);
//   * the activation tiles of a phase are requested once a grid-wide counter says that every CTA has
//     finished the phase before (a bounded wait on a global counter, not a kernel boundary);
//   * two TMEM accumulators alternate, so the epilogue of one unit overlaps the MMAs of the next;
//   * the epilogue works straight from the accumulator (thread = output feature), never touching
//     the ring, so the producer is never blocked by it.
// Split-K: every split writes its partial tile, then reduces its own share of the tile's rows (in
// split order, so the sum does not depend on timing) and applies the fused epilogue to them.  The
// per-tile arrival counters are zero at launch and are not reset.
#pragma once

#include "gemm_tc.cuh"

namespace bita {

constexpr int CH_MAX_PHASES = 4;
constexpr int CH_XCHG_TOKENS = 8;          // rows exchanged through shared memory at a time

struct ChainMaps {
  CUtensorMap a0[CH_MAX_PHASES];
  CUtensorMap a1[CH_MAX_PHASES];
  CUtensorMap b[CH_MAX_PHASES];
};

struct ChainParams {
  int32_t n_phases;
  int32_t tiles[CH_MAX_PHASES];
  GemmTcParams ph[CH_MAX_PHASES];          // M, n_pad, stages, tmem_cols are the same in every phase
  int32_t* phase_done;                     // [CH_MAX_PHASES] grid-wide arrival counters, zero at launch
};

// One unit of work: a (tile, split) pair of a phase and its K blocks.
struct ChainUnit {
  int tile, split, kb0, nkb;
};

__device__ __forceinline__ ChainUnit chain_unit(const GemmTcParams& p, int u) {
  ChainUnit r;
  r.tile = u / p.splits;
  r.split = u - r.tile * p.splits;
  const int kb_total = (p.K + TC_BLOCK_K - 1) / TC_BLOCK_K;
  r.kb0 = (int)((long)kb_total * r.split / p.splits);
  r.nkb = (int)((long)kb_total * (r.split + 1) / p.splits) - r.kb0;
  return r;
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Fused operation on up to 16 rows (c0 .. min(c0+16, row_end)-1) of one output feature: `v[j]` is
// the projection result of row c0+j for feature row `fr` of tile `tile`, already summed over the
// splits.  Called by all 128 epilogue threads together (it synchronises them when values cross
// warps).
__device__ __forceinline__ void chain_apply(const GemmTcParams& p, int tile, int fr, int lane, int c0, int row_end,
                                            float* v, const float* rstd_s, float* xchg) {
#pragma unroll
  for (int j = 0; j < 16; ++j) v[j] *= rstd_s[(c0 + j) & (BITA_MAX_ROWS - 1)];
  if (p.mode == EPI_STORE) {
    const int n = tile * TC_BLOCK_N + fr;
    if (n < p.N) {
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (c0 + j < row_end) p.out[(size_t)(c0 + j) * p.ldo + n] = v[j];
    }
  } else if (p.mode == EPI_RESID) {
    const int n = tile * TC_BLOCK_N + fr;
    const bool valid = n < p.N;
    const float g = valid ? bf2f(p.gain[n]) : 0.f;
    float xv[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) xv[j] = (valid && c0 + j < row_end) ? p.x[(size_t)(c0 + j) * p.N + n] : 0.f;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const bool live = valid && c0 + j < row_end;
      xv[j] += v[j];
      if (live) {
        p.x[(size_t)(c0 + j) * p.N + n] = xv[j];
        p.xhat[(size_t)(c0 + j) * p.N + n] = f2bf(xv[j] * g);
      }
      xv[j] = live ? xv[j] * xv[j] : 0.f;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
      for (int j = 0; j < 16; ++j) xv[j] += __shfl_xor_sync(0xffffffffu, xv[j], o);
    }
    if (lane == 0) {
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (c0 + j < row_end) atomicAdd(p.out_sumsq + c0 + j, sumsq_to_fixed(xv[j]));
    }
  } else if (p.mode == EPI_SWIGLU) {
    // tile rows 0..63 are gate features, rows 64..127 the matching up features
    const int f = tile * 64 + fr;
#pragma unroll
    for (int r8 = 0; r8 < 2; ++r8) {
      if (fr >= 64) {
#pragma unroll
        for (int j = 0; j < CH_XCHG_TOKENS; ++j) xchg[j * 64 + (fr - 64)] = v[r8 * 8 + j];
      }
      epi_bar();
      if (fr < 64 && f < p.F) {
#pragma unroll
        for (int j = 0; j < CH_XCHG_TOKENS; ++j) {
          const int tok = c0 + r8 * 8 + j;
          const float gt = v[r8 * 8 + j], up = xchg[j * 64 + fr];
          if (tok < row_end) p.hf[(size_t)tok * p.F + f] = f2bf(__fdividef(gt, 1.0f + __expf(-gt)) * up);
        }
      }
      epi_bar();
    }
  } else {                                                     // EPI_QKV
    const int n = tile * TC_BLOCK_N + fr;
    const int half = p.D >> 1;
    const int head = n / p.D, dd = n - head * p.D;
    const bool lo = dd < half;
    const int jr = lo ? dd : dd - half;
    const int partner = lo ? fr + half : fr - half;
    const bool valid = n < p.N;
    const bool rot = valid && head < p.H + p.H_kv;
    const int C = *p.len_ptr;
    bf16* dst = nullptr;
    size_t stride = 0;
    int t_end = row_end;
    if (valid) {
      if (head < p.H) {
        dst = p.q + (size_t)head * p.D + dd;
        stride = (size_t)p.H * p.D;
      } else {
        bf16* base = head < p.H + p.H_kv ? p.kc + (size_t)(head - p.H) * p.C_max * p.D
                                         : p.vc + (size_t)(head - p.H - p.H_kv) * p.C_max * p.D;
        dst = base + (size_t)C * p.D + dd;
        stride = p.D;
        t_end = min(row_end, p.C_max - C);                         // never write past the cache
      }
    }
#pragma unroll
    for (int r8 = 0; r8 < 2; ++r8) {
      float2 cs[CH_XCHG_TOKENS];
#pragma unroll
      for (int j = 0; j < CH_XCHG_TOKENS; ++j) {
        const int tok = c0 + r8 * 8 + j;
        xchg[j * TC_BLOCK_N + fr] = v[r8 * 8 + j];
        cs[j] = (rot && tok < t_end) ? p.rope_blk[(size_t)tok * half + jr] : make_float2(1.f, 0.f);
      }
      epi_bar();
      if (valid) {
#pragma unroll
        for (int j = 0; j < CH_XCHG_TOKENS; ++j) {
          const int tok = c0 + r8 * 8 + j;
          const float own = v[r8 * 8 + j], w = xchg[j * TC_BLOCK_N + partner];
          const float r = lo ? own * cs[j].x - w * cs[j].y : own * cs[j].x + w * cs[j].y;
          if (tok < t_end) dst[(size_t)tok * stride] = f2bf(r);
        }
      }
      epi_bar();
    }
  }
}

// ---------------------------------------------------------------------------------------------
// grid = (G), all CTAs resident together (the host sizes G from the occupancy of this kernel).
// Unit u of a phase goes to CTA u % G, so a CTA has at most ceil(units / G) units per phase.
__global__ void __launch_bounds__(TC_THREADS, 2) k_chain(const __grid_constant__ ChainMaps maps, ChainParams cp) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[16];
  __shared__ __align__(8) uint64_t bar_empty[16];
  __shared__ __align__(8) uint64_t bar_tfull[2];     // accumulator buffer b complete
  __shared__ __align__(8) uint64_t bar_tempty[2];    // accumulator buffer b read out
  __shared__ uint32_t tmem_base_slot;
  __shared__ float rstd_s[BITA_MAX_ROWS];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  const GemmTcParams& p0 = cp.ph[0];
  const int stages = p0.stages, n_pad = p0.n_pad;
  int32_t* status = p0.status;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t a_bytes = TC_BLOCK_N * TC_BLOCK_K * 2;
  const uint32_t b_bytes = (uint32_t)n_pad * TC_BLOCK_K * 2;
  const uint32_t stage_bytes = a_bytes + b_bytes;
  float* xchg = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)) + (size_t)stages * stage_bytes);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bar_tfull[b]), 1);
      mbar_init(smem_u32(&bar_tempty[b]), 128);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"((uint32_t)p0.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  if (threadIdx.x == 0) pdl_launch();
  if (threadIdx.x == 32) {
    for (int ph = 0; ph < cp.n_phases; ++ph) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.a0[ph]) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.b[ph]) : "memory");
    }
  }

  if (warp == 0) {
    // ---------------- TMA producer: one thread walks every K block of every unit of every phase
    if (lane == 0) {
      const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
      uint32_t it = 0;                                   // K blocks issued so far (ring position)
      bool ok = true;
      bool waited_pdl = false;
      for (int ph = 0; ph < cp.n_phases && ok; ++ph) {
        const GemmTcParams& p = cp.ph[ph];
        const int units = cp.tiles[ph] * p.splits;
        bool b_ready = false;                            // activations of this phase may be read
        uint32_t pend_it = 0;                            // first K block whose B tile is still owed
        int pend_u = 0, pend_k = 0;                      // its (unit, K block)
        bool pending = false;
        auto issue_b = [&](uint32_t at, int kb) {
          const int s = (int)(at % (uint32_t)stages);
          tma_load_2d(smem_base + (uint32_t)s * stage_bytes + a_bytes, &maps.b[ph], kb * TC_BLOCK_K, 0,
                      smem_u32(&bar_full[s]), pol_x);
        };
        // Phase 0 reads what the previous kernel wrote: its activations are ready after the
        // dependency wait, which blocks, so it is only taken when there is nothing left to prefetch
        // (`must`).  Later phases poll the arrival counter of the phase before.
        auto ready_now = [&](bool must) -> bool {
          if (ph == 0) {
            if (!must) return false;
            pdl_wait();
            waited_pdl = true;
            return true;
          }
          if (ld_acquire_gpu(cp.phase_done + ph - 1) < G) return false;
          asm volatile("fence.proxy.async;" ::: "memory");   // other CTAs' stores, then this thread's TMA reads
          if (!waited_pdl) { pdl_wait(); waited_pdl = true; }
          return true;
        };
        // B tiles owed for K blocks [pend..it): walk the same (unit, K block) order
        auto flush_pending = [&](int u_now, int k_now) {
          int u = pend_u, k = pend_k;
          uint32_t at = pend_it;
          while (u < u_now || (u == u_now && k < k_now)) {
            const ChainUnit cu = chain_unit(p, u);
            issue_b(at, cu.kb0 + k);
            ++at;
            if (++k == cu.nkb) { k = 0; u += G; }
          }
          pending = false;
        };
        for (int u = cta; u < units && ok; u += G) {
          const ChainUnit cu = chain_unit(p, u);
          const int row_a = p.dual ? cu.tile * 64 : cu.tile * TC_BLOCK_N;
          for (int k = 0; k < cu.nkb && ok; ++k) {
            const int s = (int)(it % (uint32_t)stages);
            const uint32_t par = ((it / (uint32_t)stages) & 1u) ^ 1u;
            const uint32_t empty = smem_u32(&bar_empty[s]);
            if (it >= (uint32_t)stages) {
              if (!b_ready && pending) {
                // Ring full of weight tiles that still wait for their activations: nothing frees
                // a stage until those arrive, so wait for the phase barrier here (bounded).
                unsigned long long t0 = 0;
                uint32_t spin = 0;
                while (!mbar_try_wait(empty, par)) {
                  if (ready_now(true)) { b_ready = true; flush_pending(u, k); break; }
                  if ((++spin & 63u) == 0) {
                    const unsigned long long now = global_ns();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > TC_WAIT_LIMIT_NS) { ok = false; break; }
                  }
                }
                if (!ok) { atomicExch(status, BITA_ERR_TIMEOUT); break; }
              }
              ok = mbar_wait(empty, par, status);
              if (!ok) break;
            }
            const uint32_t full = smem_u32(&bar_full[s]);
            const uint32_t sa = smem_base + (uint32_t)s * stage_bytes;
            const int kx = (cu.kb0 + k) * TC_BLOCK_K;
            mbar_expect_tx(full, stage_bytes);
            if (p.dual) {
              tma_load_2d(sa, &maps.a0[ph], kx, row_a, full, pol_w);
              tma_load_2d(sa + a_bytes / 2, &maps.a1[ph], kx, row_a, full, pol_w);
            } else {
              tma_load_2d(sa, &maps.a0[ph], kx, row_a, full, pol_w);
            }
            if (!b_ready) b_ready = ready_now(false);
            if (b_ready) {
              if (pending) flush_pending(u, k);
              issue_b(it, cu.kb0 + k);
            } else if (!pending) {
              pending = true;
              pend_it = it;
              pend_u = u;
              pend_k = k;
            }
            ++it;
          }
        }
        // weights of this phase all requested; activations still owed?
        if (ok && pending) {
          unsigned long long t0 = 0;
          uint32_t spin = 0;
          while (!ready_now(true)) {
            if ((++spin & 63u) == 0) {
              const unsigned long long now = global_ns();
              if (t0 == 0) t0 = now;
              else if (now - t0 > TC_WAIT_LIMIT_NS) { ok = false; break; }
            }
          }
          if (ok) {
            // flush up to the end of this CTA's units of the phase
            int u_end = cta;
            while (u_end < units) u_end += G;
            flush_pending(u_end, 0);
          } else {
            atomicExch(status, BITA_ERR_TIMEOUT);
          }
        }
      }
      if (!waited_pdl) pdl_wait();
      if (!ok) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);        // let the copies in flight land
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: same walk; accumulator buffers alternate between units
    if (lane == 0) {
      const uint32_t idesc = umma_idesc(n_pad);
      uint32_t it = 0, uc = 0;
      bool ok = true;
      for (int ph = 0; ph < cp.n_phases && ok; ++ph) {
        const GemmTcParams& p = cp.ph[ph];
        const int units = cp.tiles[ph] * p.splits;
        for (int u = cta; u < units && ok; u += G) {
          const ChainUnit cu = chain_unit(p, u);
          const uint32_t buf = uc & 1u;
          ok = mbar_wait(smem_u32(&bar_tempty[buf]), ((uc >> 1) & 1u) ^ 1u, status);   // buffer read out
          if (!ok) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * (uint32_t)n_pad;
          for (int k = 0; k < cu.nkb && ok; ++k) {
            const int s = (int)(it % (uint32_t)stages);
            ok = mbar_wait(smem_u32(&bar_full[s]), (it / (uint32_t)stages) & 1u, status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t sa = smem_base + (uint32_t)s * stage_bytes;
            const uint64_t da = umma_smem_desc(sa), db = umma_smem_desc(sa + a_bytes);
#pragma unroll
            for (int kk = 0; kk < TC_BLOCK_K / TC_UMMA_K; ++kk)
              umma_bf16(d_tmem, da + (uint64_t)(2 * kk), db + (uint64_t)(2 * kk), idesc, (k > 0 || kk > 0) ? 1u : 0u);
            umma_commit(smem_u32(&bar_empty[s]));
            ++it;
          }
          if (ok) umma_commit(smem_u32(&bar_tfull[buf]));
          ++uc;
        }
      }
    }
  } else {
    // ---------------- epilogue warps: thread = output feature of the tile
    const int lg = warp & 3;                                   // TMEM lane group this warp may read
    const int fr = lg * 32 + lane;
    const int tid_e = threadIdx.x - 64;
    pdl_wait();
    uint32_t uc = 0;
    bool ok = true;
    for (int ph = 0; ph < cp.n_phases; ++ph) {
      const GemmTcParams& p = cp.ph[ph];
      const int units = cp.tiles[ph] * p.splits;
      bool first = true;
      for (int u = cta; u < units; u += G) {
        const ChainUnit cu = chain_unit(p, u);
        const uint32_t buf = uc & 1u;
        if (ok) ok = mbar_wait(smem_u32(&bar_tfull[buf]), (uc >> 1) & 1u, status);
        tc_fence_after();
        if (first) {
          // everything the phase before produced is visible from here on (the producer has seen the
          // counter complete; this acquire makes it hold for this thread too)
          if (ph > 0) {
            unsigned long long t0 = 0;
            uint32_t spin = 0;
            while (ok && ld_acquire_gpu(cp.phase_done + ph - 1) < G) {
              if ((++spin & 63u) == 0) {
                const unsigned long long now = global_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > TC_WAIT_LIMIT_NS) { ok = false; atomicExch(status, BITA_ERR_TIMEOUT); }
              }
            }
          }
          for (int i = tid_e; i < BITA_MAX_ROWS; i += 128)
            rstd_s[i] = (p.in_sumsq && i < p.M && ok) ? rstd_from_sumsq(p.in_sumsq[i], p.norm_d, p.norm_eps) : 1.0f;
          epi_bar();
          first = false;
        }
        const uint32_t taddr = tmem_base + ((uint32_t)(lg * 32) << 16) + buf * (uint32_t)n_pad;
        if (p.splits == 1) {
          for (int c = 0; c < n_pad; c += 16) {
            float v[16];
            if (ok) {
              tmem_ld16(taddr + (uint32_t)c, v);
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j) v[j] = 0.f;
            }
            if (c + 16 >= n_pad) {                             // accumulator read out: the MMAs may reuse it
              tc_fence_before();
              mbar_arrive(smem_u32(&bar_tempty[buf]));
            }
            chain_apply(p, cu.tile, fr, lane, c, p.M, v, rstd_s, xchg);
          }
        } else {
          const size_t tile_elems = (size_t)p.M * TC_BLOCK_N;
          float* part_tile = p.part + (size_t)cu.tile * p.splits * tile_elems;
          float* dst = part_tile + (size_t)cu.split * tile_elems;
          for (int c = 0; c < n_pad; c += 16) {
            float v[16];
            if (ok) {
              tmem_ld16(taddr + (uint32_t)c, v);
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j) v[j] = 0.f;
            }
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (c + j < p.M) dst[(c + j) * TC_BLOCK_N + fr] = v[j];
          }
          tc_fence_before();
          mbar_arrive(smem_u32(&bar_tempty[buf]));
          __threadfence();
          epi_bar();
          if (tid_e == 0) atomicAdd(p.tile_counters + cu.tile, 1);
          // Every split of the tile reduces its own share of the rows once all partial tiles are
          // there: the other splits run on resident CTAs that reach this point without waiting
          // for this one (units are taken in (tile, split) order), so the wait is short and bounded.
          {
            unsigned long long t0 = 0;
            uint32_t spin = 0;
            while (ok && ld_acquire_gpu(p.tile_counters + cu.tile) < p.splits) {
              if ((++spin & 63u) == 0) {
                const unsigned long long now = global_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > TC_WAIT_LIMIT_NS) { ok = false; atomicExch(status, BITA_ERR_TIMEOUT); }
              }
            }
          }
          const int r_begin = (int)((long)p.M * cu.split / p.splits);
          const int r_end = (int)((long)p.M * (cu.split + 1) / p.splits);
          const int chunk = p.splits > 4 ? 8 : 16;               // at most 64 loads in flight per thread
          for (int c = r_begin; c < r_end; c += chunk) {
            const int c_end = min(r_end, c + chunk);
            float v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = 0.f;
            for (int q0 = 0; q0 < p.splits; q0 += 4) {
              float t[4][16];
#pragma unroll
              for (int rr = 0; rr < 4; ++rr) {
                const float* src = part_tile + (size_t)(q0 + rr) * tile_elems + fr;
#pragma unroll
                for (int j = 0; j < 16; ++j)
                  t[rr][j] = (ok && q0 + rr < p.splits && c + j < c_end) ? __ldcg(src + (c + j) * TC_BLOCK_N) : 0.f;
              }
#pragma unroll
              for (int rr = 0; rr < 4; ++rr) {                   // split order: fixed summation order
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] += t[rr][j];
              }
            }
            chain_apply(p, cu.tile, fr, lane, c, c_end, v, rstd_s, xchg);
          }
        }
        ++uc;
      }
      if (ph + 1 < cp.n_phases) {
        // this CTA's share of the phase is written (and will be read by TMA): tell the grid
        asm volatile("fence.proxy.async;" ::: "memory");
        __threadfence();
        epi_bar();
        if (tid_e == 0) atomicAdd(cp.phase_done + ph, 1);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p0.tmem_cols)
                 : "memory");
  }
}

}  // namespace bita
