// Small-M weight-streaming projection on the 5th-generation tensor cores (sm_100a).
//
//   Y[m][n] = sum_k X[m][k] * W[n][k]      X: bf16 [M][K] (M <= BITA_MAX_ROWS rows of the packed block)
//                                           W: bf16 [N][K] (a weight matrix, read exactly once)
//
// The roles are swapped with respect to a textbook GEMM: 128 weight rows are the MMA's M dimension
// (TMEM lanes) and the block's rows, padded to a multiple of 16, are its N dimension (TMEM
// columns).  Each CTA owns one tile of 128 output features and a contiguous range of 64-wide K
// blocks (split-K); it streams its weight tiles through a ring of TMA-filled, 128-byte-swizzled
// shared-memory stages, one elected thread issues tcgen05.mma into a TMEM accumulator, and four
// epilogue warps read the accumulator back with tcgen05.ld.  With split-K every split stores its
// partial tile in an L2-resident exchange buffer and counts itself in on a per-tile counter; once
// all splits of the tile are in, each of them sums an equal share of the tile's rows over the
// partial tiles, always in split order - every output is a fixed-order sum (deterministic, and
// independent of how many other rows the block holds) - and applies the fused operation to those
// rows.  The splits of a launch run in one wave (the host sizes the grid so) and none waits before
// its own partial tile is published, so the wait ends; it is bounded all the same.  Fused
// operations: plain fp32 store; SwiGLU ("dual" mode builds the 128-row weight tile from 64 gate
// rows and the 64 matching up rows, so both halves of a product sit in the same tile); rotary
// embedding with the q rows going to a bf16 buffer and the k/v rows straight into the KV cache;
// residual add with the next RMSNorm's input and row statistics.
//
// Programmatic dependent launch: the weight tiles of the first ring fill are requested before
// the kernel waits for its predecessor, so HBM stays busy across the kernel boundary.
//
// Every wait (mbarrier, split counter) is bounded: when the bound is hit the kernel raises the
// status word, lets its copies land, frees its TMEM and returns.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace bita {

constexpr int TC_BLOCK_N = 128;   // weight rows per tile (MMA M)
constexpr int TC_BLOCK_K = 64;    // bf16 elements per K block = 128 bytes = one swizzle row
constexpr int TC_UMMA_K = 16;
constexpr int TC_THREADS = 192;   // warp 0: TMA, warp 1: MMA + TMEM, warps 2..5: epilogue
constexpr int TC_MAX_TILES = 2048;          // tiles a launch with split-K may have (one arrival counter each)
constexpr unsigned long long TC_WAIT_LIMIT_NS = 2000000000ull;   // default bound of a device-side wait: 2 s

enum GemmEpilogue : int32_t {
  EPI_STORE = 0,    // out[m][n] = y                                   (fp32)
  EPI_SWIGLU = 1,   // dual tile: hf[m][f] = silu(gate) * up            (bf16)
  EPI_QKV = 2,      // rotary embedding, q -> bf16 buffer, k/v -> cache (bf16)
  EPI_RESID = 3,    // x[m][n] += y; xhat = bf16(x * gain); row sums of x^2 for the next RMSNorm
  EPI_HEAD = 4,     // LM head: per row, the tile's best entries as ordered keys (and the fp32 logits when asked for)
};

// Selection key of a logit: larger key = earlier in the order (value descending, token id ascending).
// The value's bits are mapped so that unsigned comparison follows the float order; a NaN never wins.
__device__ __forceinline__ unsigned long long select_key(float v, int id) {
  uint32_t b = __float_as_uint(v);
  b = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  if (!(v == v)) b = 0u;
  return ((unsigned long long)b << 32) | (uint32_t)(0xFFFFFFFFu - (uint32_t)id);
}
__device__ __forceinline__ float select_key_value(unsigned long long key) {
  uint32_t b = (uint32_t)(key >> 32);
  b = (b & 0x80000000u) ? (b & 0x7FFFFFFFu) : ~b;
  return __uint_as_float(b);
}
__device__ __forceinline__ int select_key_id(unsigned long long key) {
  return (int)(0xFFFFFFFFu - (uint32_t)(key & 0xFFFFFFFFull));
}

// RMSNorm is split between producer and consumer so that it needs no pass of its own: the
// projection that updates the residual stream x also writes xhat = bf16(x * gain) and adds its
// tile's share of sum(x^2) per row into a fixed-point accumulator (integer atomics: the sum does
// not depend on arrival order); the projection that consumes xhat multiplies its result by
// rstd = 1 / sqrt(sum / d + eps) per row, which is the same thing since the projection is linear.
constexpr float SUMSQ_SCALE = 268435456.0f;      // 2^28 fixed-point units per 1.0

__device__ __forceinline__ float rstd_from_sumsq(unsigned long long fx, int d, float eps) {
  const float ss = (float)((double)fx * (1.0 / 268435456.0));
  return rsqrtf(ss / (float)d + eps);
}
__device__ __forceinline__ unsigned long long sumsq_to_fixed(float v) {
  return __double2ull_rn((double)v * 268435456.0);
}

struct GemmTcParams {
  int32_t M;             // valid rows of X
  int32_t rows_per_seq;  // the block holds M / rows_per_seq sequences, sequence-major
  int32_t N;             // output features (for masking the last tile)
  int32_t K;
  int32_t n_pad;         // MMA N: rows of X padded to a multiple of 16
  int32_t stages;
  int32_t stg_rows;      // splits == 1: rows of the tile staged in shared memory at a time (a multiple of 96, or M)
  int32_t splits;        // split-K factor = gridDim.y
  int32_t dual;          // 1: tile = 64 rows of map A0 + 64 rows of map A1 (wide instance: 128 + 128)
  int32_t n_vtiles;      // wide instance: 128-feature "virtual" tiles of the whole launch (a CTA finishes two)
  int32_t tmem_cols;     // power of two >= max(32, n_pad)
  int32_t mode;          // GemmEpilogue
  int32_t* status;       // device status word (sticky error flag)
  unsigned long long wait_ns;   // bound of every device-side wait of the launch
  float* part;           // split-K exchange buffer [tiles][splits][M][128] fp32 (splits > 1)
  int32_t* tile_counters;  // [tiles] arrivals per tile; they only ever count up: a launch adds `splits` to each of them
  int32_t arrive_target;   // value of a tile's counter once all splits of THIS launch are in (wraps; compared as a difference)
  // row scale of the input (RMSNorm statistics of the rows of X), or null: y *= rstd(row)
  const unsigned long long* in_sumsq;
  int32_t norm_d;
  float norm_eps;
  // EPI_STORE, EPI_HEAD (null in EPI_HEAD: the logits are not kept)
  float* out;            // fp32 [M][ldo]
  int32_t ldo;
  // EPI_HEAD: cand[row][tile][BITA_MAX_TOPK] = the best sel_k(row) keys of the tile's 128 logits, best first
  unsigned long long* cand;
  const int32_t* row_kind;   // [M] RowKind: mask rows keep k_max entries, all others one (their argmax)
  int32_t k_max;
  // EPI_SWIGLU
  bf16* hf;              // bf16 [M][F]
  int32_t F;
  // EPI_RESID
  float* x;              // fp32 [M][N] residual stream, updated in place
  bf16* xhat;            // bf16 [M][N] = x * gain
  const bf16* gain;      // bf16 [N] gain of the RMSNorm that follows
  unsigned long long* out_sumsq;   // [M] fixed-point sum of x^2 per row (zeroed by the pass's first kernel)
  // EPI_QKV
  bf16* q;               // bf16 [M][H][D]
  bf16* kc;              // this layer's key cache   [H_kv][C_max][D]
  bf16* vc;              // this layer's value cache
  const float2* rope_blk;  // (cos, sin) [row][D/2] for the block's position ids
  const int32_t* len_ptr;  // cache length C of the block's first sequence (device); the next sequence's `len_stride` ints on
  int32_t len_stride;
  long long seq_stride;    // elements between the cache slabs of consecutive sequences (kc, vc point at the first one's)
  int32_t H, H_kv, D, C_max;
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait; false = gave up (status word raised).
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ int ld_acquire_gpu(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t* status,
                                          unsigned long long limit_ns = TC_WAIT_LIMIT_NS) {
  unsigned long long t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63u) == 63u) {
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) break;
    }
  }
  atomicExch(status, BITA_ERR_TIMEOUT);
  return false;
}

__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}

// 2-D tiled TMA load global -> shared (no multicast), completion on an mbarrier.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar), "l"(policy)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);          // start address, 16-byte units
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset: next group of 8 rows
  d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                         // layout: 128-byte swizzle
  return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive on an mbarrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// Wide TMEM access: n consecutive 32-bit columns of this thread's lane as 32-column instructions
// issued back to back, with ONE wait for all of them (a wait per instruction costs a round trip each).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr + 0u)
      : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, float* v) {
  uint32_t r[64];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%64];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%65];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr + 0u), "r"(taddr + 32u)
      : "memory");
#pragma unroll
  for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld96(uint32_t taddr, float* v) {
  uint32_t r[96];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%96];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%97];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%64, %65, %66, %67, %68, %69, %70, %71, %72, %73, %74, %75, %76, %77, %78, %79, %80, %81, %82, %83, %84, %85, %86, %87, %88, %89, %90, %91, %92, %93, %94, %95}, [%98];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63]), "=r"(r[64]), "=r"(r[65]), "=r"(r[66]), "=r"(r[67]), "=r"(r[68]), "=r"(r[69]), "=r"(r[70]), "=r"(r[71]), "=r"(r[72]), "=r"(r[73]), "=r"(r[74]), "=r"(r[75]), "=r"(r[76]), "=r"(r[77]), "=r"(r[78]), "=r"(r[79]), "=r"(r[80]), "=r"(r[81]), "=r"(r[82]), "=r"(r[83]), "=r"(r[84]), "=r"(r[85]), "=r"(r[86]), "=r"(r[87]), "=r"(r[88]), "=r"(r[89]), "=r"(r[90]), "=r"(r[91]), "=r"(r[92]), "=r"(r[93]), "=r"(r[94]), "=r"(r[95])
      : "r"(taddr + 0u), "r"(taddr + 32u), "r"(taddr + 64u)
      : "memory");
#pragma unroll
  for (int i = 0; i < 96; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};\n\t"
      "tcgen05.wait::st.sync.aligned;"
      :
      : "r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])), "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])), "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}
__device__ __forceinline__ void tmem_st64(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33};\n\t"
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%1], {%34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63, %64, %65};\n\t"
      "tcgen05.wait::st.sync.aligned;"
      :
      : "r"(taddr + 0u), "r"(taddr + 32u), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])), "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])), "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31])), "r"(__float_as_uint(v[32])), "r"(__float_as_uint(v[33])), "r"(__float_as_uint(v[34])), "r"(__float_as_uint(v[35])), "r"(__float_as_uint(v[36])), "r"(__float_as_uint(v[37])), "r"(__float_as_uint(v[38])), "r"(__float_as_uint(v[39])), "r"(__float_as_uint(v[40])), "r"(__float_as_uint(v[41])), "r"(__float_as_uint(v[42])), "r"(__float_as_uint(v[43])), "r"(__float_as_uint(v[44])), "r"(__float_as_uint(v[45])), "r"(__float_as_uint(v[46])), "r"(__float_as_uint(v[47])), "r"(__float_as_uint(v[48])), "r"(__float_as_uint(v[49])), "r"(__float_as_uint(v[50])), "r"(__float_as_uint(v[51])), "r"(__float_as_uint(v[52])), "r"(__float_as_uint(v[53])), "r"(__float_as_uint(v[54])), "r"(__float_as_uint(v[55])), "r"(__float_as_uint(v[56])), "r"(__float_as_uint(v[57])), "r"(__float_as_uint(v[58])), "r"(__float_as_uint(v[59])), "r"(__float_as_uint(v[60])), "r"(__float_as_uint(v[61])), "r"(__float_as_uint(v[62])), "r"(__float_as_uint(v[63]))
      : "memory");
}
// ---------------------------------------------------------------------------------------------
// Fused operation of a projection on rows [t0, t0 + cnt) of a tile, by all warps of the CTA.  A
// thread handles 4 consecutive features (quad = lane) of one row at a time; the warps take rows
// round-robin, RB rows of a warp per batch so that their loads fly together.  Partner features of
// the rotary embedding and of SwiGLU sit 64 (or 32) features away, i.e. 16 (or 8) lanes, and are
// exchanged with a warp shuffle.
//   SU == 0: the tile is complete in shared memory (`recv`, row-major [cnt][128] fp32).
//   SU  > 0: the tile is the sum of p.splits partial tiles in the exchange buffer (`part_tile`,
//            split-major).  A thread first requests everything that does not depend on the other
//            splits (residual rows, rotary factors), then `all_in()` (called by every thread of the
//            CTA, exactly once) waits for the splits, then the thread sums its quads over the
//            partial tiles, always in split order, SU loads per row in flight.
template <int RB, int SU, typename AllIn>
__device__ __forceinline__ void fused_epilogue(const GemmTcParams& p, const float* recv, const float* part_tile,
                                               size_t tile_elems, const float* rstd_s, int tile, int n_tiles, int t0,
                                               int cnt, int warp, int lane, AllIn all_in) {
  constexpr int NW = TC_THREADS / 32;
  const int n4 = tile * TC_BLOCK_N + 4 * lane;               // first output feature of the quad
  float g4[4] = {1.f, 1.f, 1.f, 1.f};
  if (p.mode == EPI_RESID && n4 + 3 < p.N) {
    const uint2 gv = *reinterpret_cast<const uint2*>(p.gain + n4);
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gv.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gv.y));
    g4[0] = a.x; g4[1] = a.y; g4[2] = b.x; g4[3] = b.y;
  }
  // EPI_QKV: which head this quad belongs to
  const int half = p.mode == EPI_QKV ? p.D >> 1 : 2;
  const int sh = half >> 2;                                  // partner quad is `sh` lanes away (16 or 8)
  const int head = p.mode == EPI_QKV ? n4 / p.D : 0, dd = p.mode == EPI_QKV ? n4 - head * p.D : 0;
  const bool lo = dd < half;
  const int jr = lo ? dd : dd - half;
  const bool rot = p.mode == EPI_QKV && n4 < p.N && head < p.H + p.H_kv;
  const bool in_n = n4 + 3 < p.N;
  const float sg = lo ? -1.f : 1.f;

  // every warp runs the same number of batches (the wait below holds a CTA-wide barrier)
  for (int b0 = 0; b0 < cnt || (SU > 0 && b0 == 0); b0 += NW * RB) {
    const int tb = b0 + warp;
    // phase A: every load of the batch (global operands, partial sums, row scales)
    float4 g0[RB], g1[RB], acc[RB];
    float rs[RB];
    bool live[RB];
#pragma unroll
    for (int u = 0; u < RB; ++u) {
      const int tl = tb + NW * u;
      live[u] = tl < cnt;
      const int tlc = live[u] ? tl : (tb < cnt ? tb : 0);    // clamp: dead rows recompute a live row, store nothing
      const int tok = t0 + tlc;
      g0[u] = make_float4(1.f, 0.f, 1.f, 0.f);
      g1[u] = make_float4(1.f, 0.f, 1.f, 0.f);
      if (cnt > 0) {
        if (p.mode == EPI_RESID) {
          if (in_n) g0[u] = *reinterpret_cast<const float4*>(p.x + (size_t)tok * p.N + n4);
        } else if (rot) {
          g0[u] = *reinterpret_cast<const float4*>(p.rope_blk + (size_t)tok * half + jr);
          g1[u] = *reinterpret_cast<const float4*>(p.rope_blk + (size_t)tok * half + jr + 2);
        }
      }
      rs[u] = cnt > 0 ? rstd_s[tok] : 0.f;
    }
    if constexpr (SU > 0) {
      if (b0 == 0) all_in();
#pragma unroll
      for (int u = 0; u < RB; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int s0 = 0; s0 < p.splits; s0 += SU) {
        float4 v[RB][SU];
#pragma unroll
        for (int u = 0; u < RB; ++u) {
          const float4* src = reinterpret_cast<const float4*>(part_tile + (size_t)(t0 + tb + NW * u) * TC_BLOCK_N) + lane;
#pragma unroll
          for (int r = 0; r < SU; ++r)
            if (live[u] && s0 + r < p.splits) v[u][r] = __ldcg(src + (size_t)(s0 + r) * (tile_elems / 4));
        }
#pragma unroll
        for (int u = 0; u < RB; ++u) {
#pragma unroll
          for (int r = 0; r < SU; ++r)
            if (live[u] && s0 + r < p.splits) {
              acc[u].x += v[u][r].x; acc[u].y += v[u][r].y; acc[u].z += v[u][r].z; acc[u].w += v[u][r].w;
            }
        }
      }
    } else {
#pragma unroll
      for (int u = 0; u < RB; ++u) {
        const int tlc = live[u] ? tb + NW * u : (tb < cnt ? tb : 0);
        acc[u] = *reinterpret_cast<const float4*>(recv + (size_t)tlc * TC_BLOCK_N + 4 * lane);
      }
    }
#pragma unroll
    for (int u = 0; u < RB; ++u) { acc[u].x *= rs[u]; acc[u].y *= rs[u]; acc[u].z *= rs[u]; acc[u].w *= rs[u]; }

    // phase B: the fused operation, written batch-wide so that independent rows interleave
    if (p.mode == EPI_RESID) {
      float ss[RB];
#pragma unroll
      for (int u = 0; u < RB; ++u) {
        ss[u] = 0.f;
        if (in_n) {                                          // N (the model width) is a multiple of 8
          float4 xv = g0[u];
          xv.x += acc[u].x; xv.y += acc[u].y; xv.z += acc[u].z; xv.w += acc[u].w;
          ss[u] = live[u] ? xv.x * xv.x + xv.y * xv.y + xv.z * xv.z + xv.w * xv.w : 0.f;
          if (live[u]) {
            const int tok = t0 + tb + NW * u;
            *reinterpret_cast<float4*>(p.x + (size_t)tok * p.N + n4) = xv;
            uint2 pk;
            pk.x = pack_bf16x2(xv.x * g4[0], xv.y * g4[1]);
            pk.y = pack_bf16x2(xv.z * g4[2], xv.w * g4[3]);
            *reinterpret_cast<uint2*>(p.xhat + (size_t)tok * p.N + n4) = pk;
          }
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int u = 0; u < RB; ++u) ss[u] += __shfl_xor_sync(0xffffffffu, ss[u], o);
      }
      if (lane == 0) {
#pragma unroll
        for (int u = 0; u < RB; ++u)
          if (live[u]) atomicAdd(p.out_sumsq + t0 + tb + NW * u, sumsq_to_fixed(ss[u]));
      }
    } else if (p.mode == EPI_STORE || p.mode == EPI_HEAD) {
      if (p.mode == EPI_HEAD) {
        // Per row: the best entries of this tile, picked one at a time by a warp-wide maximum over
        // ordered keys (a key is unique, so "remove the winner" is an equality test).
#pragma unroll
        for (int u = 0; u < RB; ++u) {
          if (!live[u]) continue;                              // warp-uniform
          const int row = t0 + tb + NW * u;
          const int kk = p.row_kind[row % p.rows_per_seq] == ROW_MASK ? p.k_max : 1;
          unsigned long long key[4];
          const float vals[4] = {acc[u].x, acc[u].y, acc[u].z, acc[u].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) key[e] = n4 + e < p.N ? select_key(vals[e], n4 + e) : 0ull;
          unsigned long long* dst = p.cand + ((size_t)row * n_tiles + tile) * BITA_MAX_TOPK;
          for (int t = 0; t < kk; ++t) {
            unsigned long long best = max(max(key[0], key[1]), max(key[2], key[3]));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
#pragma unroll
            for (int e = 0; e < 4; ++e)
              if (key[e] == best) key[e] = 0ull;
            if (lane == 0) dst[t] = best;
          }
        }
        if (!p.out) continue;
      }
#pragma unroll
      for (int u = 0; u < RB; ++u) {
        if (!live[u]) continue;
        float* dst = p.out + (size_t)(t0 + tb + NW * u) * p.ldo + n4;
        if (in_n && (p.ldo & 3) == 0) {
          *reinterpret_cast<float4*>(dst) = acc[u];
        } else {
          if (n4 < p.N) dst[0] = acc[u].x;
          if (n4 + 1 < p.N) dst[1] = acc[u].y;
          if (n4 + 2 < p.N) dst[2] = acc[u].z;
          if (n4 + 3 < p.N) dst[3] = acc[u].w;
        }
      }
    } else if (p.mode == EPI_SWIGLU) {
      // lanes 0..15 hold gate features 4*lane.., lanes 16..31 the matching up features
      float4 up[RB];
#pragma unroll
      for (int u = 0; u < RB; ++u) {
        up[u].x = __shfl_down_sync(0xffffffffu, acc[u].x, 16);
        up[u].y = __shfl_down_sync(0xffffffffu, acc[u].y, 16);
        up[u].z = __shfl_down_sync(0xffffffffu, acc[u].z, 16);
        up[u].w = __shfl_down_sync(0xffffffffu, acc[u].w, 16);
      }
      const int f = tile * 64 + 4 * lane;
      if (lane < 16 && f < p.F) {                            // F is a multiple of 8: a quad is all in or all out
#pragma unroll
        for (int u = 0; u < RB; ++u) {
          const float h0 = __fdividef(acc[u].x, 1.0f + __expf(-acc[u].x)) * up[u].x;
          const float h1 = __fdividef(acc[u].y, 1.0f + __expf(-acc[u].y)) * up[u].y;
          const float h2 = __fdividef(acc[u].z, 1.0f + __expf(-acc[u].z)) * up[u].z;
          const float h3 = __fdividef(acc[u].w, 1.0f + __expf(-acc[u].w)) * up[u].w;
          uint2 pk;
          pk.x = pack_bf16x2(h0, h1);
          pk.y = pack_bf16x2(h2, h3);
          if (live[u]) *reinterpret_cast<uint2*>(p.hf + (size_t)(t0 + tb + NW * u) * p.F + f) = pk;
        }
      }
    } else {                                                 // EPI_QKV
      // partner values: the other half of the same head
      float4 w[RB];
#pragma unroll
      for (int u = 0; u < RB; ++u) {
        w[u].x = __shfl_xor_sync(0xffffffffu, acc[u].x, sh);
        w[u].y = __shfl_xor_sync(0xffffffffu, acc[u].y, sh);
        w[u].z = __shfl_xor_sync(0xffffffffu, acc[u].z, sh);
        w[u].w = __shfl_xor_sync(0xffffffffu, acc[u].w, sh);
      }
      if (n4 < p.N) {                                        // N is a multiple of D: a quad is all in or all out
#pragma unroll
        for (int u = 0; u < RB; ++u) {
          float4 r = acc[u];
          if (rot) {
            r.x = acc[u].x * g0[u].x + sg * w[u].x * g0[u].y;
            r.y = acc[u].y * g0[u].z + sg * w[u].y * g0[u].w;
            r.z = acc[u].z * g1[u].x + sg * w[u].z * g1[u].y;
            r.w = acc[u].w * g1[u].z + sg * w[u].w * g1[u].w;
          }
          uint2 pk;
          pk.x = pack_bf16x2(r.x, r.y);
          pk.y = pack_bf16x2(r.z, r.w);
          if (!live[u]) continue;
          const int tok = t0 + tb + NW * u;
          if (head < p.H) {
            *reinterpret_cast<uint2*>(p.q + ((size_t)tok * p.H + head) * p.D + dd) = pk;
          } else {
            // row `rs` of sequence `sq` goes to slot C(sq) + rs of that sequence's cache slab
            const int sq = tok / p.rows_per_seq, rs = tok - sq * p.rows_per_seq;
            const int slot = p.len_ptr[(size_t)sq * p.len_stride] + rs;
            if (slot < p.C_max) {
              bf16* base = (head < p.H + p.H_kv ? p.kc + (size_t)(head - p.H) * p.C_max * p.D
                                                : p.vc + (size_t)(head - p.H - p.H_kv) * p.C_max * p.D) +
                           (size_t)sq * p.seq_stride;
              *reinterpret_cast<uint2*>(base + (size_t)slot * p.D + dd) = pk;
            }
          }
        }
      }
    }
  }
}

// CHUNKED: an unsplit tile whose rows do not fit the ring's memory all at once is finished
// p.stg_rows rows at a time (read back, fused operation, next rows); otherwise in one go.
// WIDE: a CTA takes 256 weight rows (two boxes of 128: consecutive rows of one matrix, or the
// matching 128 rows of a gate/up pair) against ONE activation tile: two MMAs per K step into two
// accumulators of n_pad columns (n_pad <= 256).  Half the CTAs for the same weights, and the
// activation tile is fetched once per 32 KiB of weights instead of once per 16 KiB.  The
// accumulators are finished as two "virtual" tiles of 128 features each (virtual tile 2 * tile + j),
// which is exactly what the narrow instance would have produced for them.
template <bool CHUNKED, bool WIDE>
__global__ void __launch_bounds__(TC_THREADS, 2)
k_gemm_tc(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
          const __grid_constant__ CUtensorMap map_b, GemmTcParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[16];
  __shared__ __align__(8) uint64_t bar_empty[16];
  __shared__ __align__(8) uint64_t bar_acc;
  __shared__ uint32_t tmem_base_slot;
  __shared__ float rstd_s[BITA_MAX_ROWS];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, split = blockIdx.y;
  const int kb_total = (p.K + TC_BLOCK_K - 1) / TC_BLOCK_K;
  const int kb0 = (int)((long)kb_total * split / p.splits);
  const int kb1 = (int)((long)kb_total * (split + 1) / p.splits);
  const int nkb = kb1 - kb0;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  static_assert(!(CHUNKED && WIDE), "the wide instance stages whole tiles");
  constexpr int NH = WIDE ? 2 : 1;                                      // accumulators (boxes of 128 weight rows) per CTA
  const uint32_t a_bytes = NH * TC_BLOCK_N * TC_BLOCK_K * 2;            // 16 KiB per box
  const uint32_t b_bytes = (uint32_t)p.n_pad * TC_BLOCK_K * 2;
  const uint32_t stage_bytes = a_bytes + b_bytes;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    mbar_init(smem_u32(&bar_acc), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"((uint32_t)p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (threadIdx.x == 0) pdl_launch();          // the next kernel may start its prologue
  if (threadIdx.x == 32) {                     // warm the descriptor cache while the barriers are set up
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a0) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
    if (p.dual) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a1) : "memory");
  }

  if (warp == 0) {
    // ---------------- TMA producer
    if (nkb > 0) {
      const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
      const int row_a = p.dual ? tile * 64 : tile * TC_BLOCK_N;
      auto load_a = [&](int i) {
        const int s = i % p.stages;
        const uint32_t full = smem_u32(&bar_full[s]);
        const uint32_t sa = smem_base + (uint32_t)s * stage_bytes;
        const int kx = (kb0 + i) * TC_BLOCK_K;
        mbar_expect_tx(full, stage_bytes);
        if constexpr (WIDE) {
          const int r0 = p.dual ? tile * TC_BLOCK_N : tile * 2 * TC_BLOCK_N;
          tma_load_2d(sa, &map_a0, kx, r0, full, pol_w);
          if (p.dual) tma_load_2d(sa + a_bytes / 2, &map_a1, kx, r0, full, pol_w);
          else tma_load_2d(sa + a_bytes / 2, &map_a0, kx, r0 + TC_BLOCK_N, full, pol_w);
        } else if (p.dual) {
          tma_load_2d(sa, &map_a0, kx, row_a, full, pol_w);
          tma_load_2d(sa + a_bytes / 2, &map_a1, kx, row_a, full, pol_w);
        } else {
          tma_load_2d(sa, &map_a0, kx, row_a, full, pol_w);
        }
      };
      // the activation box holds at most 256 rows: larger blocks come as two boxes of n_pad / 2 rows
      const int b_boxes = p.n_pad > 256 ? 2 : 1, b_rows = p.n_pad / b_boxes;
      auto load_b = [&](int i) {
        const int s = i % p.stages;
        for (int h = 0; h < b_boxes; ++h)
          tma_load_2d(smem_base + (uint32_t)s * stage_bytes + a_bytes + (uint32_t)(h * b_rows * TC_BLOCK_K * 2), &map_b,
                      (kb0 + i) * TC_BLOCK_K, h * b_rows, smem_u32(&bar_full[s]), pol_x);
      };
      // Weights do not depend on earlier kernels: the first ring fill requests them before the
      // kernel waits for the producer of the activations.  One lane per stage issues that first
      // fill, so the requests leave together; lane 0 alone runs the steady state.
      const int npre = nkb < p.stages ? nkb : p.stages;
      if (lane < npre) load_a(lane);
      pdl_wait();
      if (lane < npre) load_b(lane);
      __syncwarp();
      if (lane == 0) {
        bool ok = true;
        for (int i = npre; i < nkb; ++i) {
          const int s = i % p.stages;
          const uint32_t ph = (uint32_t)(i / p.stages) & 1u;
          ok = mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u, p.status, p.wait_ns);
          if (!ok) break;
          load_a(i);
          load_b(i);
        }
        if (!ok) {
          for (int i = 0; i < 64; ++i) __nanosleep(1000);    // let the copies in flight land
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0 && nkb > 0) {
      // an MMA takes at most 256 columns: larger blocks are two column halves of n_pad / 2 (a multiple of 16)
      const int halves = p.n_pad > 256 ? 2 : 1, n_half = p.n_pad / halves;
      const uint32_t idesc = umma_idesc(n_half);
      bool ok = true;
      for (int i = 0; i < nkb && ok; ++i) {
        const int s = i % p.stages;
        const uint32_t ph = (uint32_t)(i / p.stages) & 1u;
        ok = mbar_wait(smem_u32(&bar_full[s]), ph, p.status, p.wait_ns);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = smem_base + (uint32_t)s * stage_bytes;
        const uint64_t da = umma_smem_desc(sa), db = umma_smem_desc(sa + a_bytes);
        for (int h = 0; h < halves; ++h) {
          // rows [h n_half, (h + 1) n_half) of the activation tile: n_half * 128 bytes further (n_half is a multiple of 8 rows)
          const uint64_t dbh = db + (uint64_t)((h * n_half * TC_BLOCK_K * 2) >> 4);
#pragma unroll
          for (int k = 0; k < TC_BLOCK_K / TC_UMMA_K; ++k) {
            // advancing 16 elements along K = 32 bytes = 2 units of the descriptor's address field
            umma_bf16(tmem_base + (uint32_t)(h * n_half), da + (uint64_t)(2 * k), dbh + (uint64_t)(2 * k), idesc,
                      (i > 0 || k > 0) ? 1u : 0u);
            if constexpr (WIDE)     // second box of weight rows (16 KiB further), second accumulator (n_pad columns further)
              umma_bf16(tmem_base + (uint32_t)p.n_pad, da + (uint64_t)((TC_BLOCK_N * TC_BLOCK_K * 2) >> 4) + (uint64_t)(2 * k),
                        dbh + (uint64_t)(2 * k), idesc, (i > 0 || k > 0) ? 1u : 0u);
          }
        }
        umma_commit(smem_u32(&bar_empty[s]));                 // frees the stage when these MMAs are done
      }
      if (ok) umma_commit(smem_u32(&bar_acc));                // accumulator complete
    }
  }

  // ---------------- epilogue, part 1: accumulator -> staging
  // splits == 1: the tile goes to shared memory (`stg`, the pipeline stages, free once the
  //              accumulator barrier has completed), row-major [rows][128] fp32 (all M rows, or
  //              p.stg_rows at a time in the CHUNKED instance).
  // splits  > 1: every split stores its partial tile to the global exchange buffer
  //              part[tile][split][M][128] (L2-resident, overwritten by every projection) and
  //              counts itself in; once all splits of the tile are in, each of them sums an equal
  //              share of the rows over the partial tiles, always in split order, and applies
  //              the fused operation to those rows.
  float* stg = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)));
  const size_t tile_elems = (size_t)p.M * TC_BLOCK_N;
  float* part_tile = p.part + (size_t)tile * NH * p.splits * tile_elems;  // this tile's partials: [virtual tile][split]
  if (warp >= 2) {
    const int lg = warp & 3;                                   // TMEM lane group this warp may read
    const int fr = lg * 32 + lane;                             // feature row of the tile owned by this thread
    // While the main loop streams: wait for the earlier kernels (their outputs are read below, and
    // the exchange buffer was last read by an earlier projection) and fetch the per-row scales of
    // the unnormalised input rows (RMSNorm finished on the consumer side).
    pdl_wait();
    for (int i = threadIdx.x - 64; i < p.M; i += 128)
      rstd_s[i] = p.in_sumsq ? rstd_from_sumsq(p.in_sumsq[i], p.norm_d, p.norm_eps) : 1.0f;
    bool ok = true;
    if (nkb > 0) ok = mbar_wait(smem_u32(&bar_acc), 0, p.status, p.wait_ns);
    tc_fence_after();
    if constexpr (!WIDE) {
      float* dst = p.splits > 1 ? part_tile + (size_t)split * tile_elems : stg;
      ok = __all_sync(0xffffffffu, ok);                          // the TMEM loads below are warp-wide
      const uint32_t lane_addr = tmem_base + ((uint32_t)(lg * 32) << 16);
      const int c_end = CHUNKED ? min(p.n_pad, p.stg_rows) : p.n_pad;   // CHUNKED: the first rows only
      for (int c = 0; c < c_end; c += 96) {                      // up to 96 columns per TMEM round trip
        float v[96];
        const int groups = min(3, (p.n_pad - c + 31) >> 5);      // 32-column groups, inside the allocation
        if (nkb > 0 && ok) {
          if (groups == 1) tmem_ld32(lane_addr + (uint32_t)c, v);
          else if (groups == 2) tmem_ld64(lane_addr + (uint32_t)c, v);
          else tmem_ld96(lane_addr + (uint32_t)c, v);
        } else {
#pragma unroll
          for (int j = 0; j < 96; ++j) v[j] = 0.f;
        }
#pragma unroll
        for (int j = 0; j < 96; ++j)
          if (j < groups * 32 && c + j < p.M) dst[(c + j) * TC_BLOCK_N + fr] = v[j];
      }
    } else {
      ok = __all_sync(0xffffffffu, ok);                          // the TMEM loads below are warp-wide
      const uint32_t lane_addr = tmem_base + ((uint32_t)(lg * 32) << 16);
      const int c_end = CHUNKED ? min(p.n_pad, p.stg_rows) : p.n_pad;   // CHUNKED: the first rows only
#pragma unroll
      for (int hv = 0; hv < NH; ++hv) {
        // Where feature row `fr` of accumulator hv goes: virtual tile vj, column vc of its 128.  A wide
        // gate/up pair (accumulator 0 = 128 gate rows, 1 = the matching up rows) is laid out as two
        // pair tiles of 64 + 64, the layout the SwiGLU operation expects.
        int vj = hv, vc = fr;
        if (WIDE && p.dual) { vj = fr >> 6; vc = hv * 64 + (fr & 63); }
        float* dst = p.splits > 1 ? part_tile + ((size_t)vj * p.splits + split) * tile_elems : stg + (size_t)vj * tile_elems;
        for (int c = 0; c < c_end; c += 96) {                    // up to 96 columns per TMEM round trip
          float v[96];
          const int groups = min(3, (p.n_pad - c + 31) >> 5);    // 32-column groups, inside the allocation
          if (nkb > 0 && ok) {
            const uint32_t ta = lane_addr + (uint32_t)(hv * p.n_pad + c);
            if (groups == 1) tmem_ld32(ta, v);
            else if (groups == 2) tmem_ld64(ta, v);
            else tmem_ld96(ta, v);
          } else {
#pragma unroll
            for (int j = 0; j < 96; ++j) v[j] = 0.f;
          }
#pragma unroll
          for (int j = 0; j < 96; ++j)
            if (j < groups * 32 && c + j < p.M) dst[(c + j) * TC_BLOCK_N + vc] = v[j];
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  // ---------------- epilogue, part 2: reduction over the splits + fused operation, all six warps.
  // Rows of the tile this CTA finishes: all of them without a split, else an equal share, so that
  // the reduction and the fused operation of a tile are spread over all its splits.
  const int t0 = p.splits > 1 ? (int)((long)p.M * split / p.splits) : 0;
  const int cnt = (p.splits > 1 ? (int)((long)p.M * (split + 1) / p.splits) : (CHUNKED ? min(p.M, p.stg_rows) : p.M)) - t0;
  pdl_wait();
  if constexpr (!WIDE) {
    if (p.splits == 1) {
      fused_epilogue<6, 0>(p, stg, nullptr, tile_elems, rstd_s, tile, (int)gridDim.x, t0, cnt, warp, lane, [] {});
      if constexpr (CHUNKED) {
        // the remaining rows, p.stg_rows (a multiple of 96) at a time through the same staging memory
        for (int c0 = p.stg_rows; c0 < p.M; c0 += p.stg_rows) {
          const int c1 = min(c0 + p.stg_rows, p.M);
          __syncthreads();                                       // the staging rows are rewritten
          if (warp >= 2) {
            const int fr = (warp & 3) * 32 + lane;
            const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
            for (int c = c0; c < c1; c += 96) {
              float v[96];
              const int groups = min(3, (p.n_pad - c + 31) >> 5);
              if (nkb > 0) {
                if (groups == 1) tmem_ld32(lane_addr + (uint32_t)c, v);
                else if (groups == 2) tmem_ld64(lane_addr + (uint32_t)c, v);
                else tmem_ld96(lane_addr + (uint32_t)c, v);
              } else {
#pragma unroll
                for (int j = 0; j < 96; ++j) v[j] = 0.f;
              }
#pragma unroll
              for (int j = 0; j < 96; ++j)
                if (j < groups * 32 && c + j < p.M) stg[(c + j - c0) * TC_BLOCK_N + fr] = v[j];
            }
          }
          tc_fence_before();
          __syncthreads();
          fused_epilogue<6, 0>(p, stg, nullptr, tile_elems, rstd_s, tile, (int)gridDim.x, c0, c1 - c0, warp, lane, [] {});
        }
      }
    } else {
      int32_t* arrived = p.tile_counters + tile;
      if (threadIdx.x == 0) {
        __threadfence();                                         // the CTA's partial tile (ordered by the barrier above) before the count
        atomicAdd(arrived, 1);
      }
      // The splits of a tile are CTAs of one wave (the host sizes the grid so), none of which waits
      // before it has published its own partial tile: the wait ends, and it is bounded all the same.
      // The counter is never reset: the host tells each launch the value that means "all in", so no
      // split has to report that it has finished reading (the exchange buffer is next written by a
      // later kernel, which starts its own stores only after this one has completed).
      auto all_in = [&]() {
        if (threadIdx.x == 0) {
          unsigned long long w0 = 0;
          bool ok = true;
          for (uint32_t spin = 0; (int32_t)((uint32_t)ld_acquire_gpu(arrived) - (uint32_t)p.arrive_target) < 0; ++spin) {
            if ((spin & 63u) == 63u) {
              const unsigned long long now = global_ns();
              if (w0 == 0) w0 = now;
              else if (now - w0 > p.wait_ns) { ok = false; break; }
            }
          }
          if (!ok) atomicExch(p.status, BITA_ERR_TIMEOUT);
          __threadfence();
        }
        __syncthreads();
      };
      // rows per batch x loads per row in flight, sized so that a 69..128-row block takes one batch
      const int nt = (int)gridDim.x;
      if (p.splits == 2) fused_epilogue<6, 2>(p, nullptr, part_tile, tile_elems, rstd_s, tile, nt, t0, cnt, warp, lane, all_in);
      else if (p.splits == 3) fused_epilogue<4, 3>(p, nullptr, part_tile, tile_elems, rstd_s, tile, nt, t0, cnt, warp, lane, all_in);
      else if (p.splits == 4) fused_epilogue<4, 4>(p, nullptr, part_tile, tile_elems, rstd_s, tile, nt, t0, cnt, warp, lane, all_in);
      else fused_epilogue<2, 8>(p, nullptr, part_tile, tile_elems, rstd_s, tile, nt, t0, cnt, warp, lane, all_in);
    }
  } else {
    const int nt = p.n_vtiles;                                  // 128-feature tiles of the launch
    if (p.splits == 1) {
#pragma unroll
      for (int vj = 0; vj < NH; ++vj) {
        const int vt = tile * NH + vj;
        if (vt < nt) fused_epilogue<6, 0>(p, stg + (size_t)vj * tile_elems, nullptr, tile_elems, rstd_s, vt, nt, t0, cnt, warp, lane, [] {});
      }
    } else {
      int32_t* arrived = p.tile_counters + tile;
      if (threadIdx.x == 0) {
        __threadfence();                                         // the CTA's partial tile (ordered by the barrier above) before the count
        atomicAdd(arrived, 1);
      }
      // The splits of a tile are CTAs of one wave (the host sizes the grid so), none of which waits
      // before it has published its own partial tile: the wait ends, and it is bounded all the same.
      // The counter is never reset: the host tells each launch the value that means "all in", so no
      // split has to report that it has finished reading (the exchange buffer is next written by a
      // later kernel, which starts its own stores only after this one has completed).
      auto all_in = [&]() {
        if (threadIdx.x == 0) {
          unsigned long long w0 = 0;
          bool ok = true;
          for (uint32_t spin = 0; (int32_t)((uint32_t)ld_acquire_gpu(arrived) - (uint32_t)p.arrive_target) < 0; ++spin) {
            if ((spin & 63u) == 63u) {
              const unsigned long long now = global_ns();
              if (w0 == 0) w0 = now;
              else if (now - w0 > p.wait_ns) { ok = false; break; }
            }
          }
          if (!ok) atomicExch(p.status, BITA_ERR_TIMEOUT);
          __threadfence();
        }
        __syncthreads();
      };
      // rows per batch x loads per row in flight, sized so that a 69..128-row block takes one batch
      bool waited = false;
#pragma unroll
      for (int vj = 0; vj < NH; ++vj) {
        const int vt = tile * NH + vj;
        const float* pt = part_tile + (size_t)vj * p.splits * tile_elems;
        auto once = [&]() { if (!waited) { all_in(); waited = true; } };   // the tile's splits are waited for once
        if (vt >= nt) { once(); continue; }
        if (p.splits == 2) fused_epilogue<6, 2>(p, nullptr, pt, tile_elems, rstd_s, vt, nt, t0, cnt, warp, lane, once);
        else if (p.splits == 3) fused_epilogue<4, 3>(p, nullptr, pt, tile_elems, rstd_s, vt, nt, t0, cnt, warp, lane, once);
        else if (p.splits == 4) fused_epilogue<4, 4>(p, nullptr, pt, tile_elems, rstd_s, vt, nt, t0, cnt, warp, lane, once);
        else fused_epilogue<2, 8>(p, nullptr, pt, tile_elems, rstd_s, vt, nt, t0, cnt, warp, lane, once);
      }
    }
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols)
                 : "memory");
  }
}

}  // namespace bita
