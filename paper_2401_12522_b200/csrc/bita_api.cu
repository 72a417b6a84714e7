// Host side of the BiTA step library: argument checks, block plans, workspace carving and the
// launch sequence of one pass.  Every step of the pass runs in the kernels included below.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <new>
#include <tuple>
#include <vector>

#include "attention_umma.cuh"
#include "common.cuh"
#include "gemm_tc.cuh"
#include "step_kernels.cuh"

using namespace bita;

namespace {

thread_local int g_last_cuda_error = 0;

#define CU_TRY(expr)                                   \
  do {                                                 \
    cudaError_t e__ = (expr);                          \
    if (e__ != cudaSuccess) {                          \
      g_last_cuda_error = (int)e__;                    \
      return BITA_ERR_CUDA;                            \
    }                                                  \
  } while (0)

// Launch with optional thread-block cluster along y and optional programmatic dependent launch.
template <typename... P, typename... A>
int launch(cudaStream_t s, bool pdl, dim3 grid, dim3 block, size_t smem, unsigned cluster_y, void (*kernel)(P...),
           A... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[2];
  unsigned n = 0;
  if (cluster_y > 1) {
    at[n].id = cudaLaunchAttributeClusterDimension;
    at[n].val.clusterDim.x = 1;
    at[n].val.clusterDim.y = cluster_y;
    at[n].val.clusterDim.z = 1;
    ++n;
  }
  if (pdl) {
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = at;
  cfg.numAttrs = n;
  CU_TRY(cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...));
  return BITA_OK;
}

constexpr int PREFILL_CHUNK = BITA_MAX_ROWS - BITA_MAX_MASK;   // query rows per block of the first pass
constexpr size_t ALIGN = 256;

inline size_t align_up(size_t v) { return (v + ALIGN - 1) / ALIGN * ALIGN; }

// Host description of a packed block; `upload_plan` writes it into a device region and fills `dev`.
struct HostPlan {
  int M = 0, W = 0, N = 0, G = 0, n_mask = 0, k_max = 1, n_query = 0, max_depth = 0;
  int B = 1, seq0 = 0;     // sequences in the block (M = rows of one of them), first sequence
  std::vector<int32_t> row_kind, row_idx, rel_pos, parent, rank, depth, group_of;
  std::vector<uint8_t> sees_prompt;
  std::vector<uint32_t> vis;
  DevPlan dev{};
};

constexpr size_t PLAN_REGION_BYTES =
    sizeof(int32_t) * (3 * BITA_MAX_ROWS + BITA_MAX_ROWS * (BITA_MAX_ROWS / 32) + 3 * BITA_MAX_NODES +
                       (BITA_MAX_NODES + 1)) + BITA_MAX_ROWS + 1024;

// Step block (Sec. 3.2, Appendix B): root, tree nodes, G groups of n mask tokens, for each of
// `batch` sequences (the tables describe one sequence; the block repeats them sequence-major).
int build_step_plan(const bita_tree_template* t, int n_mask, int batch, HostPlan* p) {
  if (batch < 1 || batch > BITA_MAX_BATCH) return BITA_ERR_INVALID_ARG;
  if (!t || t->N < 0 || t->N > BITA_MAX_NODES || t->G < 0) return BITA_ERR_BAD_TEMPLATE;
  if (t->N > 0 && (!t->parent || !t->rank)) return BITA_ERR_BAD_TEMPLATE;
  if (t->G > 0 && !t->attach) return BITA_ERR_BAD_TEMPLATE;
  if (n_mask < 0 || n_mask > BITA_MAX_MASK) return BITA_ERR_INVALID_ARG;
  const int N = t->N, G = t->G;
  const long rows = 1L + N + (long)G * n_mask;
  if (rows * batch > BITA_MAX_ROWS) return BITA_ERR_BAD_TEMPLATE;
  p->M = (int)rows;
  p->B = batch;
  p->seq0 = 0;
  p->W = (p->M + 31) / 32;
  p->N = N;
  p->G = G;
  p->n_mask = n_mask;
  p->n_query = 0;
  p->parent.assign(t->parent, t->parent + N);
  p->rank.assign(t->rank, t->rank + N);
  p->depth.assign(N, 0);
  p->k_max = 1;
  p->max_depth = 0;
  for (int i = 0; i < N; ++i) {
    if (p->parent[i] < -1 || p->parent[i] >= i) return BITA_ERR_BAD_TEMPLATE;
    if (p->rank[i] < 0 || p->rank[i] >= BITA_MAX_TOPK) return BITA_ERR_BAD_TEMPLATE;
    p->depth[i] = p->parent[i] < 0 ? 1 : p->depth[p->parent[i]] + 1;
    if (p->depth[i] > BITA_MAX_DEPTH) return BITA_ERR_BAD_TEMPLATE;
    if (p->depth[i] > p->max_depth) p->max_depth = p->depth[i];
    if (p->rank[i] + 1 > p->k_max) p->k_max = p->rank[i] + 1;
  }
  p->group_of.assign(N + 1, -1);
  for (int g = 0; g < G; ++g) {
    const int a = t->attach[g];
    if (a < -1 || a >= N || p->group_of[a + 1] >= 0) return BITA_ERR_BAD_TEMPLATE;
    p->group_of[a + 1] = g;
  }
  const int M = p->M, W = p->W;
  p->row_kind.assign(M, ROW_MASK);
  p->row_idx.assign(M, 0);
  p->rel_pos.assign(M, 0);
  p->sees_prompt.assign(M, 0);
  p->vis.assign((size_t)M * W, 0u);
  auto set = [&](int r, int c) { p->vis[(size_t)r * W + (c >> 5)] |= 1u << (c & 31); };
  auto inherit = [&](int r, int from) {
    for (int w = 0; w < W; ++w) p->vis[(size_t)r * W + w] |= p->vis[(size_t)from * W + w];
  };
  p->row_kind[0] = ROW_ROOT;
  set(0, 0);
  for (int i = 0; i < N; ++i) {
    const int r = 1 + i;
    p->row_kind[r] = ROW_NODE;
    p->row_idx[r] = i;
    p->rel_pos[r] = p->depth[i];
    inherit(r, p->parent[i] + 1);   // the parent's row already holds root..parent
    set(r, r);
  }
  for (int g = 0; g < G; ++g) {
    const int arow = t->attach[g] + 1;
    for (int i = 0; i < n_mask; ++i) {
      const int r = 1 + N + g * n_mask + i;
      p->row_idx[r] = i;
      p->rel_pos[r] = p->rel_pos[arow] + i + 1;
      p->sees_prompt[r] = 1;
      inherit(r, arow);
      for (int j = 0; j <= i; ++j) set(r, 1 + N + g * n_mask + j);   // causal inside the group
    }
  }
  return BITA_OK;
}

// Prefill chunk (Algorithm 1, t = 1): `cnt` query tokens, causal; the last chunk is followed by
// one group of n_mask mask tokens attached to the final query token.
void build_prefill_plan(int cnt, int n_mask, bool last, int k_max, int seq, HostPlan* p) {
  const int M = cnt + (last ? n_mask : 0);
  p->M = M;
  p->B = 1;
  p->seq0 = seq;
  p->W = (M + 31) / 32;
  p->N = 0;
  p->G = last ? 1 : 0;
  p->n_mask = n_mask;
  p->k_max = k_max;
  p->n_query = cnt;
  p->max_depth = 0;
  p->parent.clear();
  p->rank.clear();
  p->depth.clear();
  p->group_of.assign(1, -1);
  p->row_kind.assign(M, ROW_QUERY);
  p->row_idx.assign(M, 0);
  p->rel_pos.assign(M, 0);
  p->sees_prompt.assign(M, 0);
  p->vis.assign((size_t)M * p->W, 0u);
  for (int r = 0; r < M; ++r) {
    p->rel_pos[r] = r;
    if (r >= cnt) {
      p->row_kind[r] = ROW_MASK;
      p->row_idx[r] = r - cnt;
      p->sees_prompt[r] = 1;
    } else {
      p->row_idx[r] = r;
    }
    for (int c = 0; c <= r; ++c) p->vis[(size_t)r * p->W + (c >> 5)] |= 1u << (c & 31);
  }
}

int upload_plan(HostPlan* p, void* region, cudaStream_t stream) {
  std::vector<uint8_t> blob(PLAN_REGION_BYTES, 0);
  size_t off = 0;
  bool overflow = false;
  auto put = [&](const void* src, size_t bytes) -> const void* {
    const size_t at = off;
    if (at + bytes > PLAN_REGION_BYTES) { overflow = true; return region; }
    if (bytes) memcpy(blob.data() + at, src, bytes);
    off = (at + bytes + 15) / 16 * 16;
    return (const uint8_t*)region + at;
  };
  DevPlan& d = p->dev;
  d.M = p->M; d.B = p->B; d.seq0 = p->seq0; d.W = p->W; d.N = p->N; d.G = p->G; d.n_mask = p->n_mask; d.k_max = p->k_max;
  d.n_query = p->n_query; d.max_depth = p->max_depth;
  d.row_kind = (const int32_t*)put(p->row_kind.data(), p->row_kind.size() * 4);
  d.row_idx = (const int32_t*)put(p->row_idx.data(), p->row_idx.size() * 4);
  d.rel_pos = (const int32_t*)put(p->rel_pos.data(), p->rel_pos.size() * 4);
  d.vis = (const uint32_t*)put(p->vis.data(), p->vis.size() * 4);
  d.parent = (const int32_t*)put(p->parent.data(), p->parent.size() * 4);
  d.rank = (const int32_t*)put(p->rank.data(), p->rank.size() * 4);
  d.depth = (const int32_t*)put(p->depth.data(), p->depth.size() * 4);
  d.group_of = (const int32_t*)put(p->group_of.data(), p->group_of.size() * 4);
  d.sees_prompt = (const uint8_t*)put(p->sees_prompt.data(), p->sees_prompt.size());
  if (overflow) return BITA_ERR_BAD_TEMPLATE;
  CU_TRY(cudaMemcpyAsync(region, blob.data(), off ? off : 16, cudaMemcpyHostToDevice, stream));
  CU_TRY(cudaStreamSynchronize(stream));
  return BITA_OK;
}

int check_dims(const bita_model_dims* m) {
  if (!m) return BITA_ERR_INVALID_ARG;
  if (m->L < 1 || m->d < 8 || m->d % 8 || m->H < 1 || m->H_kv < 1 || m->H % m->H_kv) return BITA_ERR_INVALID_ARG;
  if (m->D != 64 && m->D != 128) return BITA_ERR_INVALID_ARG;
  if (m->F < 8 || m->F % 8 || m->V < 1 || m->P < 0 || m->P > 64 || m->C_max < 1) return BITA_ERR_INVALID_ARG;
  if (!(m->rms_eps >= 0.f) || !(m->rope_theta > 0.f)) return BITA_ERR_INVALID_ARG;
  return BITA_OK;
}

// ---------------------------------------------------------------------------------------------
// Tensor-core projection: host-side planning (tensor maps, split-K, pipeline depth).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return (EncodeTiledFn)p;
  }();
  return fn;
}

// bf16 matrix [rows][K] (K contiguous) -> map with a (64 x box_rows) box, 128-byte swizzle, zero fill.
int make_map(CUtensorMap* m, const void* base, int K, int rows, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return BITA_ERR_CUDA;
  if (((uintptr_t)base & 15) || (K % 8)) return BITA_ERR_INVALID_ARG;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)TC_BLOCK_K, (cuuint32_t)box_rows};
  cuuint32_t es[2] = {1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return BITA_ERR_CUDA; }
  return BITA_OK;
}

// bf16 tensor [d2][d1][d0] (d0 contiguous, the given byte strides) -> 3-D map, 128-byte swizzle, zero fill.
int make_map3(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1,
              uint64_t stride2, uint32_t box1, uint32_t box2) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return BITA_ERR_CUDA;
  if (((uintptr_t)base & 15) || (stride1 & 15) || (stride2 & 15)) return BITA_ERR_INVALID_ARG;
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {stride1, stride2};
  cuuint32_t box[3] = {64, box1, box2};
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return BITA_ERR_CUDA; }
  return BITA_OK;
}

// One weight matrix (or a gate/up pair) as the projection kernel sees it.
struct GemmDesc {
  CUtensorMap a0, a1;
  CUtensorMap a0w, a1w;   // the same matrices with boxes of 128 rows (wide tiles); for a single matrix a0w = a0
  int max_splits = 8;
  const void *w0 = nullptr, *w1 = nullptr;
  int N = 0, K = 0, dual = 0, tiles = 0, splits = 1;
  int kind = 0;           // which set of split-arrival counters its launches count on (GemmKind)
};

// Split-K factor: as many CTAs as stay resident together (two per SM while the block is small, the
// shared-memory ring of a CTA then being half an SM's), never fewer than 4 K blocks per split.
constexpr int GEMM_MAX_CTAS = 296;       // size of the exchange buffer: two CTAs on each of up to 148 SMs
constexpr int GEMM_MAX_SPLITS = 8;
// Launches that may follow one another with different shapes count their split arrivals on sets of
// their own, so that every counter of a set moves by the same amount with every launch of its kind.
enum GemmKind { KIND_QKV = 0, KIND_O, KIND_GU, KIND_DN, KIND_HEAD, GEMM_KINDS };

// What the library remembers per device of the process: CUDA keeps function attributes and
// device properties per device, so none of this may be a process-wide flag.
constexpr int MAX_DEVICES = 64;
struct DeviceFacts {
  int sms = 0;
  bool gemm_attr = false, attn_attr = false, select_attr = false;
  void* static_scratch = nullptr;
};
DeviceFacts g_device[MAX_DEVICES];
DeviceFacts g_device_overflow;          // devices beyond MAX_DEVICES: looked up every time

DeviceFacts* device_facts() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
    g_device_overflow = DeviceFacts();
    return &g_device_overflow;
  }
  return &g_device[dev];
}

// SMs of the current device (the splits of a launch wait for one another, so a launch with splits
// never has more CTAs than the GPU holds at once); capped at what the exchange buffer is sized for.
int sm_count() {
  DeviceFacts* f = device_facts();
  if (!f->sms) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
      f->sms = v > GEMM_MAX_CTAS / 2 ? GEMM_MAX_CTAS / 2 : v;
    else
      f->sms = 1;
  }
  return f->sms;
}

int gemm_splits(int tiles, int K, int max_splits) {
  const int kb = (K + TC_BLOCK_K - 1) / TC_BLOCK_K;
  int s = 2 * sm_count() / tiles;
  if (s > kb / 4) s = kb / 4;
  if (s > max_splits) s = max_splits;
  if (s > GEMM_MAX_SPLITS) s = GEMM_MAX_SPLITS;
  if (s < 1) s = 1;
  return s;
}

int make_gemm_desc(GemmDesc* g, const void* W0, const void* W1, int N, int K, int max_splits) {
  g->K = K;
  g->dual = W1 ? 1 : 0;
  g->w0 = W0;
  g->w1 = W1;
  int rc;
  if (W1) {           // N = rows of each of the two matrices
    g->tiles = (N + 63) / 64;
    g->N = N;
    if ((rc = make_map(&g->a0, W0, K, N, 64))) return rc;
    if ((rc = make_map(&g->a1, W1, K, N, 64))) return rc;
    if ((rc = make_map(&g->a0w, W0, K, N, TC_BLOCK_N))) return rc;
    if ((rc = make_map(&g->a1w, W1, K, N, TC_BLOCK_N))) return rc;
  } else {
    g->tiles = (N + TC_BLOCK_N - 1) / TC_BLOCK_N;
    g->N = N;
    if ((rc = make_map(&g->a0, W0, K, N, TC_BLOCK_N))) return rc;
    g->a1 = g->a0;
    g->a0w = g->a0;
    g->a1w = g->a0;
  }
  g->max_splits = max_splits;
  if (g->tiles > TC_MAX_TILES) return BITA_ERR_INVALID_ARG;
  g->splits = gemm_splits(g->tiles, K, max_splits);
  return BITA_OK;
}

// Padded row count of a block as the MMA sees it: a multiple of 16; past 256 rows a multiple of 32,
// so that each of the two column halves is a multiple of 16.
inline int pad16(int m) { return m <= 16 ? 16 : (m <= 256 ? (m + 15) / 16 * 16 : (m + 31) / 32 * 32); }

// Blocks of up to this many padded rows run two CTAs per SM (two accumulators of up to 256 columns
// share the SM's tensor memory, two rings its shared memory); larger ones one CTA per SM.
constexpr int TWO_PER_SM_MAX_ROWS = 256;

// How a projection is launched for a block of n_pad padded rows (M valid ones).
struct GemmPlan {
  bool wide = false;      // 256 weight rows per CTA (two accumulators), see k_gemm_tc
  bool chunked = false;   // unsplit tile finished stg_rows rows at a time
  int tiles = 0;          // gridDim.x
  int splits = 1;         // gridDim.y
  int stages = 2;
  int stg_rows = 0;
  int tmem_cols = 32;
  size_t smem = 0;
};

// 0 = never, 1 = wherever the shapes allow, -1 (default) = where it pays: launches whose narrow
// tiles would need a second wave of CTAs.
int wide_policy() {
  static const int v = [] {
    const char* e = getenv("BITA_WIDE_TILES");
    return e ? atoi(e) : -1;
  }();
  return v;
}

GemmPlan plan_gemm(const GemmDesc& g, int n_pad, int M) {
  GemmPlan pl;
  const int sms = sm_count();
  const int kb = (g.K + TC_BLOCK_K - 1) / TC_BLOCK_K;
  const size_t extra = 1024;                                   // alignment slack
  // ---- narrow: 128 weight rows per CTA
  auto narrow = [&]() {
    GemmPlan n;
    n.tiles = g.tiles;
    n.splits = g.splits;
    // with one CTA per SM a split only pays while all its CTAs fit in one wave
    if (n_pad > TWO_PER_SM_MAX_ROWS && g.tiles * n.splits > sms) n.splits = sms / g.tiles > 0 ? sms / g.tiles : 1;
    int cols = 32;
    while (cols < n_pad) cols <<= 1;
    n.tmem_cols = cols;
    const size_t stage = (size_t)TC_BLOCK_N * TC_BLOCK_K * 2 + (size_t)n_pad * TC_BLOCK_K * 2;
    // Two CTAs per SM take half the shared memory each: 4 ring stages up to 96 rows, 3 up to 160, 2 beyond.
    const bool two_per_sm = n_pad <= TWO_PER_SM_MAX_ROWS && g.tiles * n.splits > sms;
    const size_t budget = (two_per_sm ? 110 : 220) * 1024;
    int stages = (int)((budget - extra) / stage);
    if (stages > 10) stages = 10;
    if (stages < 2) stages = 2;
    n.stages = stages;
    // an unsplit tile is finished from a staging copy in the ring's memory: all rows at once if they fit, else 96 at a time
    const int fit = (int)((size_t)stages * stage / ((size_t)TC_BLOCK_N * 4));
    n.stg_rows = fit >= M ? M : fit / 96 * 96;
    n.chunked = n.splits == 1 && n.stg_rows < M;
    n.smem = stages * stage + extra;
    return n;
  };
  pl = narrow();
  const int policy = wide_policy();
  if (policy == 0 || n_pad > 256 || g.tiles < 2) return pl;
  // ---- wide: 256 weight rows per CTA, half the CTAs
  GemmPlan w;
  w.wide = true;
  w.tiles = (g.tiles + 1) / 2;
  const bool small = n_pad <= 128;                             // two accumulators of <= 128 columns: two CTAs per SM possible
  int s = (small ? 2 * sms : sms) / w.tiles;
  if (s > kb / 4) s = kb / 4;
  if (s > g.max_splits) s = g.max_splits;
  if (s > GEMM_MAX_SPLITS) s = GEMM_MAX_SPLITS;
  if (s < 1) s = 1;
  w.splits = s;
  int cols = 32;
  while (cols < 2 * n_pad) cols <<= 1;
  w.tmem_cols = cols;
  const size_t stage = (size_t)2 * TC_BLOCK_N * TC_BLOCK_K * 2 + (size_t)n_pad * TC_BLOCK_K * 2;
  const bool two_per_sm = small && w.tiles * s > sms;
  const size_t budget = (two_per_sm ? 110 : 220) * 1024;
  int stages = (int)((budget - extra) / stage);
  if (stages > 10) stages = 10;
  if (stages < 2) return pl;
  w.stages = stages;
  w.stg_rows = M;
  if (s == 1 && (size_t)stages * stage < (size_t)2 * M * TC_BLOCK_N * 4) return pl;   // both accumulators are staged whole
  if (w.tiles * s > (small ? 2 * sms : sms)) return pl;        // the wide launch itself must be one wave
  w.smem = stages * stage + extra;
  if (policy == 1) return w;
  // default: only where the narrow launch does not fit the GPU at once
  const int slots = n_pad <= TWO_PER_SM_MAX_ROWS ? 2 * sms : sms;
  return pl.tiles * pl.splits > slots ? w : pl;
}

int effective_splits(const GemmDesc& g, int n_pad, int M) { return plan_gemm(g, n_pad, M).splits; }

// Launch: X bf16 (first M rows valid) times the described weights; `p` carries the epilogue.
int launch_gemm_tc(const GemmDesc& g, const CUtensorMap& map_b, int n_pad, int M, GemmTcParams p, bool pdl,
                   cudaStream_t stream) {
  DeviceFacts* facts = device_facts();
  if (!facts->gemm_attr) {
    CU_TRY(cudaFuncSetAttribute(k_gemm_tc<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024));
    CU_TRY(cudaFuncSetAttribute(k_gemm_tc<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024));
    CU_TRY(cudaFuncSetAttribute(k_gemm_tc<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024));
    facts->gemm_attr = true;
  }
  if (!p.wait_ns) p.wait_ns = TC_WAIT_LIMIT_NS;
  const GemmPlan pl = plan_gemm(g, n_pad, M);
  p.M = M; p.N = g.N; p.K = g.K; p.n_pad = n_pad; p.dual = g.dual;
  p.n_vtiles = g.tiles;
  if (p.rows_per_seq < 1) p.rows_per_seq = M;
  p.tmem_cols = pl.tmem_cols;
  p.stg_rows = pl.stg_rows;
  if (p.stg_rows < 1) return BITA_ERR_INVALID_ARG;
  p.splits = pl.splits;
  p.stages = pl.stages;
  const dim3 grid(pl.tiles, pl.splits);
  if (pl.wide)
    return launch(stream, pdl, grid, dim3(TC_THREADS), pl.smem, 1, k_gemm_tc<false, true>, g.a0w, g.a1w, map_b, p);
  if (pl.chunked)
    return launch(stream, pdl, grid, dim3(TC_THREADS), pl.smem, 1, k_gemm_tc<true, false>, g.a0, g.a1, map_b, p);
  return launch(stream, pdl, grid, dim3(TC_THREADS), pl.smem, 1, k_gemm_tc<false, false>, g.a0, g.a1, map_b, p);
}


// Attention launch shape: row tiles (one CTA takes one tile of 128 query rows, or two when the block
// has more than 128 rows), and key slices.  The slices of a (sequence,
// head, row tile) form a thread-block cluster; the slice count is the largest cluster size whose
// clusters all fit the GPU at once (one CTA per SM; concurrent clusters seen on a B200: 74 of size
// 2, 45 of 3, 33 of 4, 22 of 6, 15 of 8).  More clusters than that would still be correct (they
// run in waves), just not faster.
void attn_shape(int H, int B, int M, int* row_tiles, int* splits) {
  const int rt = (M + 2 * AU_ROWS - 1) / (2 * AU_ROWS);       // a CTA takes up to two tiles of 128 rows
  const int groups = H * B * rt;
  static const int size[5] = {8, 6, 4, 3, 2}, fit[5] = {15, 22, 33, 45, 74};
  int s = 1;
  for (int i = 0; i < 5; ++i)
    if (groups <= fit[i]) { s = size[i]; break; }
  *row_tiles = rt; *splits = s;
}

int attn_splits(int H, int B, int M) {
  int rt, s;
  attn_shape(H, B, M, &rt, &s);
  return s;
}

// Long caches: key slices for the workspace route (partial results in global memory, merged by a
// second kernel), where the slice count is free: the CTAs of such a launch run in waves of one per
// SM, and the count is chosen so that the waves come out even.  Cost of a choice in units of "one
// CTA works through one chunk of 128 keys": waves(groups * S) * ceil(chunks / S), plus the traffic of
// the partial results (M rows of D + 2 floats per group and slice, written and read once) at the rate
// the GPU streams keys and values (one chunk = 64 KiB per SM).  Returns 0 when the cluster shape is
// within 5 % of the best (short caches always: launch latency matters more there).
constexpr int ATTN_MAX_WS_SLICES = 64;
int attn_balanced_slices(int H, int B, int M, int D, int C_max) {
  int rt, s0;
  attn_shape(H, B, M, &rt, &s0);
  const int sms = sm_count();
  const long groups = (long)H * B * rt;
  const long chunks = (C_max + AU_KEYS - 1) / AU_KEYS + 1;
  if (chunks < 128) return 0;
  auto waves = [&](long ctas) { return (ctas + sms - 1) / sms; };
  const double part_unit = (double)M * (D + 2) * 4 * 2 / ((double)sms * 2 * AU_KEYS * D * 2);   // per group and slice
  const double base = (double)waves(groups * s0) * ((chunks + s0 - 1) / s0);
  double best = base;
  int best_s = 0;
  for (int s = 1; s <= ATTN_MAX_WS_SLICES; ++s) {
    if (chunks / s < 4) break;
    const double cost = (double)waves(groups * s) * ((chunks + s - 1) / s) + (s > 1 ? part_unit * groups * s : 0.0) + 2.0;
    if (cost < best * 0.95 && (best_s == 0 || cost < best)) { best = cost; best_s = s; }
  }
  return best_s;
}

// Device buffers of a context, carved from the caller's workspace.
struct Buffers {
  float* x; bf16* xn; bf16* q; bf16* att; bf16* hf; unsigned long long* cand; unsigned long long* sumsq;
  int32_t* sel_id; float* sel_val; int32_t* pos; int32_t* row_token; float* part_ml; float* part_acc; float* gemm_part; int32_t* gemm_cnt;
  float2* rope_tab; float2* rope_blk; DevState* state; DevRecord* rec; void* plan_step; void* plan_prefill;
  int32_t* query_tokens; int32_t* tree_in;
};

size_t carve(const bita_model_dims& m, uint8_t* base, Buffers* b) {
  size_t off = 0;
  auto take = [&](size_t bytes) -> void* {
    void* p = base ? base + off : nullptr;
    off += align_up(bytes);
    return p;
  };
  const size_t R = BITA_MAX_ROWS;
  const size_t wide = (size_t)m.d > (size_t)m.H * m.D ? m.d : (size_t)m.H * m.D;
  Buffers t{};
  t.x = (float*)take(R * m.d * 4);
  t.xn = (bf16*)take(R * wide * 2);
  t.q = (bf16*)take(R * m.H * m.D * 2);
  t.att = (bf16*)take(R * m.H * m.D * 2);
  t.sumsq = (unsigned long long*)take((size_t)(2 * m.L + 1) * R * 8);
  t.hf = (bf16*)take(R * (size_t)m.F * 2);
  t.cand = (unsigned long long*)take(R * (size_t)((m.V + TC_BLOCK_N - 1) / TC_BLOCK_N) * BITA_MAX_TOPK * 8);
  t.sel_id = (int32_t*)take(R * BITA_MAX_TOPK * 4);
  t.sel_val = (float*)take(R * BITA_MAX_TOPK * 4);
  t.pos = (int32_t*)take(R * 4);
  t.row_token = (int32_t*)take(R * 4);
  const size_t S = 8;                        // upper bound of attn_splits
  t.part_ml = (float*)take((size_t)m.H * S * R * 2 * 4);
  t.part_acc = (float*)take((size_t)m.H * S * R * m.D * 4);
  t.gemm_part = (float*)take((size_t)2 * GEMM_MAX_CTAS * R * TC_BLOCK_N * 4);   // a wide CTA leaves two partial tiles
  t.gemm_cnt = (int32_t*)take((size_t)2 * GEMM_KINDS * TC_MAX_TILES * 4);
  t.rope_tab = (float2*)take((size_t)(m.C_max + 64) * (m.D / 2) * sizeof(float2));
  t.rope_blk = (float2*)take(R * (size_t)(m.D / 2) * sizeof(float2));
  t.state = (DevState*)take(sizeof(DevState) * BITA_MAX_BATCH);      // one per sequence
  t.rec = (DevRecord*)take(sizeof(DevRecord) * BITA_MAX_BATCH);
  t.plan_step = take(PLAN_REGION_BYTES);
  t.plan_prefill = take(PLAN_REGION_BYTES);
  t.query_tokens = (int32_t*)take(PREFILL_CHUNK * 4);
  t.tree_in = (int32_t*)take((size_t)BITA_MAX_ROWS * 4);               // [B][N] tree tokens of a step, B * N < rows
  if (b) *b = t;
  return off;
}

}  // namespace

struct bita_ctx {
  bita_model_dims m;
  int n_mask;
  std::vector<const void*> wqkv, wo, wg, wu, wd, g_attn, g_ffn, prompt_k, prompt_v;
  const void *tok_emb, *mask_emb, *g_final, *lm_head;
  cudaStream_t stream;
  Buffers b;
  HostPlan step_plan, prefill_plan;
  int B;                    // sequences decoded together (1 for bita_init)
  DevRecord* rec_host;      // pinned, one record per sequence
  std::vector<int> len_upper;       // per sequence: upper bound of the device-side cache length
  std::vector<char> prefilled;      // per sequence
  float* dbg;
  int launches;
  std::vector<GemmDesc> d_qkv, d_o, d_gu, d_dn;
  GemmDesc d_head;
  std::map<std::tuple<const void*, int, int>, CUtensorMap> act_maps;   // (buffer, K, padded rows) -> map
  std::map<std::tuple<const void*, const void*, const void*, const void*, int, int, int, int>, AttnMaps> attn_map_cache;
  bool pdl;                             // programmatic dependent launch between the kernels of a pass
  uint32_t split_arrivals[2 * GEMM_KINDS];  // what every counter of a set has reached once the launches so far are done
  unsigned long long wait_ns;           // bound of every device-side wait
  int last_rows;                        // rows of the most recent pass (what the debug buffer holds)

  // optional per-family event timing
  bool timing;
  std::vector<cudaEvent_t> ev;          // pairs (start, stop)
  std::vector<int> ev_family;           // timing: family of the run of launches that follows event i (-1 = end)
  std::vector<int> ev_count;            // launches in that run
};

namespace {

// Timing marks: one event wherever the kernel family changes, so that a run of consecutive
// launches of one family (e.g. O, gate/up, down and the next q/k/v projection) is timed as it
// runs in an untimed pass, with each kernel's first weight tiles requested during its predecessor's
// tail.  Families: 0 projections, 1 attention, 2 everything else, -1 closes the pass.
void mark(bita_ctx* c, int family) {
  if (!c->timing) return;
  if (c->ev_family.empty() || c->ev_family.back() != family) {
    const size_t i = c->ev_family.size();
    if (i >= c->ev.size()) {
      cudaEvent_t e = nullptr;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      c->ev.push_back(e);
    }
    cudaEventRecord(c->ev[i], c->stream);
    c->ev_family.push_back(family);
    c->ev_count.push_back(0);
  }
  if (family >= 0) c->ev_count.back() += 1;
}

// Projection of the first M rows of an activation buffer (BITA_MAX_ROWS rows allocated).
int gemm(bita_ctx* c, const GemmDesc& g, const bf16* X, int M, GemmTcParams p) {
  const int n_pad = pad16(M);
  auto key = std::make_tuple((const void*)X, g.K, n_pad);
  auto it = c->act_maps.find(key);
  if (it == c->act_maps.end()) {
    CUtensorMap m;
    int rc = make_map(&m, X, g.K, BITA_MAX_ROWS, n_pad > 256 ? n_pad / 2 : n_pad);
    if (rc) return rc;
    it = c->act_maps.emplace(key, m).first;
  }
  p.status = &c->b.state->status;
  p.wait_ns = c->wait_ns;
  p.part = c->b.gemm_part;
  {
    // wide and narrow launches of a kind count on sets of their own (they cover different tile ranges)
    const GemmPlan pl = plan_gemm(g, n_pad, M);
    const int set = g.kind + (pl.wide ? GEMM_KINDS : 0);
    p.tile_counters = c->b.gemm_cnt + (size_t)set * TC_MAX_TILES;
    if (pl.splits > 1) c->split_arrivals[set] += (uint32_t)pl.splits;
    p.arrive_target = (int32_t)c->split_arrivals[set];
  }
  mark(c, 0);
  int rc = launch_gemm_tc(g, it->second, n_pad, M, p, c->pdl, c->stream);
  c->launches++;
  return rc;
}

GemmTcParams epi_store(float* out, int ldo) {
  GemmTcParams p{};
  p.mode = EPI_STORE; p.out = out; p.ldo = ldo;
  return p;
}

// Tensor maps of an attention call; `cache` (may be null) keeps them across calls with the same
// buffers and shapes.
using AttnMapKey = std::tuple<const void*, const void*, const void*, const void*, int, int, int, int>;
int attn_maps(const AttnArgs& a, std::map<AttnMapKey, AttnMaps>* cache, AttnMaps* out) {
  const AttnMapKey key{a.q, a.k, a.v, a.prompt_k, a.B * a.M, a.H * 1024 + a.H_kv, a.C_max, a.P * 1024 + a.D};
  if (cache) {
    auto it = cache->find(key);
    if (it != cache->end()) { *out = it->second; return BITA_OK; }
  }
  const uint64_t D = a.D, row = D * 2;
  int rc;
  if ((rc = make_map3(&out->q, a.q, D, a.H, (uint64_t)a.B * a.M, row, row * a.H, 1, AU_ROWS))) return rc;
  if ((rc = make_map3(&out->k, a.k, D, a.C_max, (uint64_t)a.B * a.H_kv, row, row * a.C_max, AU_KEYS, 1))) return rc;
  if ((rc = make_map3(&out->v, a.v, D, a.C_max, (uint64_t)a.B * a.H_kv, row, row * a.C_max, AU_KEYS, 1))) return rc;
  if (a.P > 0 && a.prompt_k && a.prompt_v) {
    if ((rc = make_map3(&out->pk, a.prompt_k, D, a.P, a.H_kv, row, row * a.P, AU_KEYS, 1))) return rc;
    if ((rc = make_map3(&out->pv, a.prompt_v, D, a.P, a.H_kv, row, row * a.P, AU_KEYS, 1))) return rc;
  } else {
    out->pk = out->k;
    out->pv = out->v;
  }
  if (cache) cache->emplace(key, *out);
  return BITA_OK;
}

// Fills the launch-shape fields of `a` (row_tiles, S, scale) and launches the slices (and the merge
// kernel where the slices cannot merge themselves).
// `route`: ATTN_ROUTE_AUTO merges the slices inside a thread-block cluster and falls back to the
// workspace route only when that launch form is refused; ATTN_ROUTE_WORKSPACE always sends the
// partial results through a.part_ml / a.part_acc and the merge kernel.
enum { ATTN_ROUTE_AUTO = 0, ATTN_ROUTE_WORKSPACE = 1 };
int g_attention_route = ATTN_ROUTE_AUTO;      // process-wide diagnostic switch (bita_set_attention_route)

int launch_attention(AttnArgs a, bool pdl, cudaStream_t s, int* n_launched, std::map<AttnMapKey, AttnMaps>* cache,
                     int route = -1, int ws_slices = 0) {
  if (route < 0) route = g_attention_route;
  attn_shape(a.H, a.B, a.M, &a.row_tiles, &a.S);
  if (ws_slices > 0) {                   // the caller's workspace holds that many slices: even waves, merge kernel
    a.S = ws_slices;
    if (ws_slices > 1) route = ATTN_ROUTE_WORKSPACE;
  }
  AttnMaps maps;
  {
    int rc = attn_maps(a, cache, &maps);
    if (rc) return rc;
  }
  a.scale_log2 = 1.4426950408889634f / sqrtf((float)a.D);
  const int RT = a.M > AU_ROWS ? 2 : 1;                          // row tiles per CTA
  const size_t tile = (size_t)(a.D / 64) * AU_ATOM;
  const size_t smem = (RT + 4) * tile + 2 * AU_ATOM + 1024;       // Q (RT tiles), 2 x (K, V), P
  DeviceFacts* facts = device_facts();
  if (!a.wait_ns) a.wait_ns = TC_WAIT_LIMIT_NS;
  if (!facts->attn_attr) {
    CU_TRY(cudaFuncSetAttribute(k_attn_umma<128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 202 * 1024));
    CU_TRY(cudaFuncSetAttribute(k_attn_umma<64, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 202 * 1024));
    CU_TRY(cudaFuncSetAttribute(k_attn_umma<128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
    CU_TRY(cudaFuncSetAttribute(k_attn_umma<64, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
    facts->attn_attr = true;
  }
  dim3 g1(a.H, a.S, a.B * a.row_tiles), g2(a.M, a.H, a.B);
  auto run = [&](unsigned cluster_y) {
    if (a.D == 128)
      return RT == 2 ? launch(s, pdl, g1, dim3(AU_THREADS), smem, cluster_y, k_attn_umma<128, 2>, maps, a)
                     : launch(s, pdl, g1, dim3(AU_THREADS), smem, cluster_y, k_attn_umma<128, 1>, maps, a);
    return RT == 2 ? launch(s, pdl, g1, dim3(AU_THREADS), smem, cluster_y, k_attn_umma<64, 2>, maps, a)
                   : launch(s, pdl, g1, dim3(AU_THREADS), smem, cluster_y, k_attn_umma<64, 1>, maps, a);
  };
  if (n_launched) *n_launched = 1;
  if (a.S == 1) return run(1);
  int rc;
  if (route != ATTN_ROUTE_WORKSPACE) {
    a.cluster = 1;
    rc = run((unsigned)a.S);
    if (rc == BITA_OK) return rc;
    // The cluster launch was refused: the slices leave their partial results in global memory
    // and a second kernel merges them.
    (void)cudaGetLastError();
  }
  a.cluster = 0;
  if (n_launched) *n_launched = 2;
  if ((rc = run(1))) return rc;
  return a.D == 128 ? launch(s, pdl, g2, dim3(64), 0, 1, k_attn_merge<128>, a)
                    : launch(s, pdl, g2, dim3(32), 0, 1, k_attn_merge<64>, a);
}

// The layer stack over one packed block, then (optionally) the LM head and selection.
int run_block(bita_ctx* c, bita_kv* kv, const HostPlan& hp, const int32_t* tree_dev, bool want_logits) {
  const bita_model_dims& m = c->m;
  const DevPlan& P = hp.dev;
  const int M = P.M * P.B;                                   // rows of the block: P.B sequences of P.M rows
  cudaStream_t s = c->stream;
  Buffers& b = c->b;
  c->ev_family.clear();
  c->ev_count.clear();
  c->last_rows = M;
  mark(c, 2);
  const size_t seq_kv = (size_t)m.H_kv * kv->C_max * m.D;      // one sequence's slab of a layer
  const size_t layer_kv = seq_kv * c->B;                       // cache layout [L][B][H_kv][C_max][D]
  const size_t block_kv = seq_kv * P.seq0;                     // the block's first sequence within a layer
  const DevState* st0 = b.state + P.seq0;
  const bool pdl = c->pdl;
  int rc;
  const int n_slots = 2 * m.L + 1;
  auto slot = [&](int i) { return b.sumsq + (size_t)i * BITA_MAX_ROWS; };
  if ((rc = launch(s, pdl, dim3(M), dim3(256), 0, 1, k_embed, P, (const DevState*)b.state, tree_dev,
                   (const int32_t*)b.query_tokens, (const bf16*)c->tok_emb, (const bf16*)c->mask_emb, m.d, m.V, b.x,
                   b.pos, b.row_token, (const float2*)b.rope_tab, m.D / 2, b.rope_blk, (const bf16*)c->g_attn[0],
                   b.xn, b.sumsq, n_slots)))
    return rc;
  c->launches += 1;
  auto with_norm = [&](GemmTcParams p, int in_slot) {
    p.in_sumsq = slot(in_slot);
    p.norm_d = m.d;
    p.norm_eps = m.rms_eps;
    return p;
  };
  auto epi_resid = [&](const void* gain, int out_slot) {
    GemmTcParams p{};
    p.mode = EPI_RESID; p.x = b.x; p.xhat = b.xn; p.gain = (const bf16*)gain; p.out_sumsq = slot(out_slot);
    return p;
  };
  struct ProjOp { const GemmDesc* g; const bf16* X; GemmTcParams p; };
  auto op_qkv = [&](int l) {
    GemmTcParams p{};
    p.mode = EPI_QKV; p.q = b.q;
    p.kc = (bf16*)kv->k + (size_t)l * layer_kv + block_kv; p.vc = (bf16*)kv->v + (size_t)l * layer_kv + block_kv;
    p.rope_blk = b.rope_blk; p.len_ptr = &st0->len; p.len_stride = (int32_t)(sizeof(DevState) / 4);
    p.seq_stride = (long long)seq_kv; p.H = m.H; p.H_kv = m.H_kv; p.D = m.D; p.C_max = kv->C_max;
    return ProjOp{&c->d_qkv[l], b.xn, with_norm(p, 2 * l)};       // attention RMSNorm scale + q/k/v + RoPE + cache write
  };
  auto op_o = [&](int l) {   // output projection + residual add; leaves x * g_ffn and the row statistics
    return ProjOp{&c->d_o[l], b.att, epi_resid(c->g_ffn[l], 2 * l + 1)};
  };
  auto op_gu = [&](int l) {  // FFN RMSNorm scale + gate/up projection + SwiGLU
    GemmTcParams p{};
    p.mode = EPI_SWIGLU; p.hf = b.hf; p.F = m.F;
    return ProjOp{&c->d_gu[l], b.xn, with_norm(p, 2 * l + 1)};
  };
  auto op_dn = [&](int l) {  // down projection + residual add; leaves x * gain of the next norm
    const void* g_next = l + 1 < m.L ? c->g_attn[l + 1] : c->g_final;
    return ProjOp{&c->d_dn[l], b.hf, epi_resid(g_next, 2 * l + 2)};
  };
  auto single = [&](ProjOp o) { o.p.rows_per_seq = P.M; return gemm(c, *o.g, o.X, M, o.p); };
  for (int l = 0; l < m.L; ++l) {
    bf16* kc = (bf16*)kv->k + (size_t)l * layer_kv + block_kv;
    bf16* vc = (bf16*)kv->v + (size_t)l * layer_kv + block_kv;
    if ((rc = single(op_qkv(l)))) return rc;
    AttnArgs a{};
    a.q = b.q; a.k = kc; a.v = vc; a.vis = P.vis; a.prompt_k = (const bf16*)c->prompt_k[l];
    a.prompt_v = (const bf16*)c->prompt_v[l]; a.sees_prompt = P.sees_prompt; a.ctx_len = &st0->len;
    a.ctx_len_stride = (int32_t)(sizeof(DevState) / 4);
    a.vis_batch_stride = 0; a.sp_batch_stride = 0; a.out = b.att; a.part_ml = b.part_ml; a.part_acc = b.part_acc;
    a.B = P.B; a.M = P.M; a.W = P.W; a.H = m.H; a.H_kv = m.H_kv; a.D = m.D; a.P = m.P; a.C_max = kv->C_max;
    a.status = &b.state->status;
    a.wait_ns = c->wait_ns;
    {
      mark(c, 1);
      int n = 0;
      if ((rc = launch_attention(a, pdl, s, &n, &c->attn_map_cache))) return rc;
      c->launches += n;
    }
    if ((rc = single(op_o(l)))) return rc;
    if ((rc = single(op_gu(l)))) return rc;
    if ((rc = single(op_dn(l)))) return rc;
    if (c->dbg)
      CU_TRY(cudaMemcpyAsync(c->dbg + (size_t)l * BITA_MAX_ROWS * m.d, b.x, (size_t)M * m.d * 4,
                             cudaMemcpyDeviceToDevice, s));
  }
  if (want_logits) {
    // LM head with the first half of the selection in its epilogue; the logits themselves are kept
    // only when a debug buffer asks for them.
    GemmTcParams hp{};
    hp.mode = EPI_HEAD;
    hp.out = c->dbg ? c->dbg + (size_t)m.L * BITA_MAX_ROWS * m.d : nullptr;
    hp.ldo = m.V;
    hp.cand = b.cand;
    hp.row_kind = P.row_kind;
    hp.k_max = P.k_max;
    hp.rows_per_seq = P.M;
    if ((rc = gemm(c, c->d_head, b.xn, M, with_norm(hp, 2 * m.L)))) return rc;
    mark(c, 2);
    if ((rc = launch(s, pdl, dim3(M), dim3(256), 0, 1, k_select_merge, P, (const unsigned long long*)b.cand,
                     c->d_head.tiles, b.sel_id, b.sel_val)))
      return rc;
    c->launches += 1;
  }
  mark(c, -1);
  CU_TRY(cudaGetLastError());
  return BITA_OK;
}

void fill_out(const DevRecord* r, bita_step_out* out) {
  out->status = r->status;
  out->n_out = r->n_out;
  out->new_len = r->new_len;
  memcpy(out->out_tokens, r->out_tokens, sizeof(out->out_tokens));
  memcpy(out->accepted_idx, r->accepted_idx, sizeof(out->accepted_idx));
  memcpy(out->next_tree, r->next_tree, sizeof(out->next_tree));
}

}  // namespace

extern "C" {

int bita_workspace_bytes_batch(const bita_model_dims* dims, const bita_tree_template* tmpl, int n_mask, int32_t batch,
                               size_t* out_bytes) {
  if (!out_bytes) return BITA_ERR_INVALID_ARG;
  int rc = check_dims(dims);
  if (rc) return rc;
  HostPlan p;
  rc = build_step_plan(tmpl, n_mask, batch, &p);
  if (rc) return rc;
  *out_bytes = carve(*dims, nullptr, nullptr);
  return BITA_OK;
}

int bita_workspace_bytes(const bita_model_dims* dims, const bita_tree_template* tmpl, int n_mask, size_t* out_bytes) {
  return bita_workspace_bytes_batch(dims, tmpl, n_mask, 1, out_bytes);
}

int bita_init_batch(bita_ctx** out, const bita_model_dims* dims, const bita_weights* w, const bita_tree_template* tmpl,
                    int n_mask, int32_t batch, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!out || !w || !workspace) return BITA_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = check_dims(dims);
  if (rc) return rc;
  if (!w->tok_emb || !w->g_final || !w->lm_head || !w->wqkv || !w->wo || !w->wg || !w->wu || !w->wd || !w->g_attn ||
      !w->g_ffn)
    return BITA_ERR_INVALID_ARG;
  if (n_mask > 0 && !w->mask_emb) return BITA_ERR_INVALID_ARG;
  if (dims->P > 0 && (!w->prompt_k || !w->prompt_v)) return BITA_ERR_INVALID_ARG;
  bita_ctx* c = new (std::nothrow) bita_ctx();
  if (!c) return BITA_ERR_INVALID_ARG;
  rc = build_step_plan(tmpl, n_mask, batch, &c->step_plan);
  if (rc) { delete c; return rc; }
  if (((uintptr_t)workspace % ALIGN) || workspace_bytes < carve(*dims, nullptr, nullptr)) {
    delete c;
    return BITA_ERR_WORKSPACE;
  }
  c->m = *dims;
  c->n_mask = n_mask;
  c->B = batch;
  c->stream = (cudaStream_t)cuda_stream;
  c->tok_emb = w->tok_emb; c->mask_emb = w->mask_emb; c->g_final = w->g_final; c->lm_head = w->lm_head;
  const int L = dims->L;
  auto cp = [&](std::vector<const void*>& v, const void* const* src, bool need) -> bool {
    v.assign(L, nullptr);
    if (!src) return !need;
    for (int l = 0; l < L; ++l) { v[l] = src[l]; if (need && !src[l]) return false; }
    return true;
  };
  bool ok = cp(c->wqkv, w->wqkv, true) && cp(c->wo, w->wo, true) && cp(c->wg, w->wg, true) && cp(c->wu, w->wu, true) &&
            cp(c->wd, w->wd, true) && cp(c->g_attn, w->g_attn, true) && cp(c->g_ffn, w->g_ffn, true) &&
            cp(c->prompt_k, w->prompt_k, dims->P > 0) && cp(c->prompt_v, w->prompt_v, dims->P > 0);
  if (!ok) { delete c; return BITA_ERR_INVALID_ARG; }
  carve(*dims, (uint8_t*)workspace, &c->b);
  c->rec_host = nullptr;
  c->dbg = nullptr;
  c->launches = 0;
  c->timing = false;
  c->pdl = getenv("BITA_NO_PDL") == nullptr;
  c->wait_ns = TC_WAIT_LIMIT_NS;
  c->last_rows = 0;

  c->prefilled.assign(batch, 0);
  c->len_upper.assign(batch, 0);
  auto fail = [&](int code) { if (c->rec_host) cudaFreeHost(c->rec_host); delete c; return code; };
  if (cudaMallocHost((void**)&c->rec_host, sizeof(DevRecord) * BITA_MAX_BATCH) != cudaSuccess) return fail(BITA_ERR_CUDA);
  memset(c->rec_host, 0, sizeof(DevRecord) * BITA_MAX_BATCH);
  // rotary table in double precision: angle = pos * theta^(-2j/D)
  {
    const int half = dims->D / 2, npos = dims->C_max + 64;
    std::vector<float2> tab((size_t)npos * half);
    std::vector<double> inv(half);
    for (int j = 0; j < half; ++j) inv[j] = pow((double)dims->rope_theta, -2.0 * j / dims->D);
    for (int p = 0; p < npos; ++p)
      for (int j = 0; j < half; ++j) {
        const double ang = (double)p * inv[j];
        tab[(size_t)p * half + j] = make_float2((float)cos(ang), (float)sin(ang));
      }
    if (cudaMemcpyAsync(c->b.rope_tab, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice, c->stream) !=
            cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess)
      return fail(BITA_ERR_CUDA);
  }
  {
    const int nqkv = (dims->H + 2 * dims->H_kv) * dims->D;
    c->d_qkv.resize(L); c->d_o.resize(L); c->d_gu.resize(L); c->d_dn.resize(L);
    for (int l = 0; l < L; ++l) {
      if ((rc = make_gemm_desc(&c->d_qkv[l], c->wqkv[l], nullptr, nqkv, dims->d, 8))) return fail(rc);
      if ((rc = make_gemm_desc(&c->d_o[l], c->wo[l], nullptr, dims->d, dims->H * dims->D, 8))) return fail(rc);
      if ((rc = make_gemm_desc(&c->d_gu[l], c->wg[l], c->wu[l], dims->F, dims->d, 8))) return fail(rc);
      if ((rc = make_gemm_desc(&c->d_dn[l], c->wd[l], nullptr, dims->d, dims->F, 8))) return fail(rc);
      c->d_qkv[l].kind = KIND_QKV; c->d_o[l].kind = KIND_O; c->d_gu[l].kind = KIND_GU; c->d_dn[l].kind = KIND_DN;
    }
    if ((rc = make_gemm_desc(&c->d_head, c->lm_head, nullptr, dims->V, dims->d, 1))) return fail(rc);
    c->d_head.kind = KIND_HEAD;
  }
  rc = upload_plan(&c->step_plan, c->b.plan_step, c->stream);
  if (rc) return fail(rc);
  if (cudaMemsetAsync(c->b.gemm_cnt, 0, (size_t)2 * GEMM_KINDS * TC_MAX_TILES * 4, c->stream) != cudaSuccess) return fail(BITA_ERR_CUDA);
  for (int k = 0; k < 2 * GEMM_KINDS; ++k) c->split_arrivals[k] = 0;
  k_reset_state<<<BITA_MAX_BATCH, 128, 0, c->stream>>>(c->b.state);
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return fail(BITA_ERR_CUDA);
  *out = c;
  return BITA_OK;
}

int bita_init(bita_ctx** out, const bita_model_dims* dims, const bita_weights* w, const bita_tree_template* tmpl,
              int n_mask, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return bita_init_batch(out, dims, w, tmpl, n_mask, 1, workspace, workspace_bytes, cuda_stream);
}

int bita_batch(const bita_ctx* c) { return c ? c->B : BITA_ERR_INVALID_ARG; }

int bita_reset(bita_ctx* c, bita_kv* kv) {
  if (!c || !kv) return BITA_ERR_INVALID_ARG;
  // a pass that gave up on a wait may have left split counters half way
  CU_TRY(cudaMemsetAsync(c->b.gemm_cnt, 0, (size_t)2 * GEMM_KINDS * TC_MAX_TILES * 4, c->stream));
  for (int k = 0; k < 2 * GEMM_KINDS; ++k) c->split_arrivals[k] = 0;
  k_reset_state<<<BITA_MAX_BATCH, 128, 0, c->stream>>>(c->b.state);
  CU_TRY(cudaStreamSynchronize(c->stream));
  c->prefilled.assign(c->B, 0);
  c->len_upper.assign(c->B, 0);
  return BITA_OK;
}

int bita_rewind_seq(bita_ctx* c, bita_kv* kv, int32_t seq, int32_t new_len, int32_t last_token) {
  if (!c || !kv || seq < 0 || seq >= c->B) return BITA_ERR_INVALID_ARG;
  if (!c->prefilled[seq]) return BITA_ERR_NOT_PREFILLED;
  if (new_len < 0 || new_len > c->len_upper[seq] || last_token < 0 || last_token >= c->m.V) return BITA_ERR_INVALID_ARG;
  k_set_state<<<1, 128, 0, c->stream>>>(c->b.state + seq, new_len, last_token);
  CU_TRY(cudaGetLastError());
  c->len_upper[seq] = new_len;
  return BITA_OK;
}

int bita_rewind(bita_ctx* c, bita_kv* kv, int32_t new_len, int32_t last_token) {
  return bita_rewind_seq(c, kv, 0, new_len, last_token);
}

int bita_prefill_seq(bita_ctx* c, bita_kv* kv, int32_t seq, const int32_t* tokens, int32_t count, bita_step_out* out) {
  if (!c || !kv || !kv->k || !kv->v || !tokens || count < 1 || seq < 0 || seq >= c->B) return BITA_ERR_INVALID_ARG;
  if (kv->C_max != c->m.C_max) return BITA_ERR_INVALID_ARG;
  for (int i = 0; i < count; ++i)
    if (tokens[i] < 0 || tokens[i] >= c->m.V) return BITA_ERR_INVALID_ARG;
  if ((long)c->len_upper[seq] + count + c->n_mask > kv->C_max) return BITA_ERR_KV_FULL;
  c->launches = 0;
  // Equal blocks, as few as the row limit allows: every block streams all the weights once.
  int blocks_left = (count + PREFILL_CHUNK - 1) / PREFILL_CHUNK;
  for (int done = 0; done < count; --blocks_left) {
    const int cnt = (count - done + blocks_left - 1) / blocks_left;
    const bool last = done + cnt == count;
    build_prefill_plan(cnt, c->n_mask, last, c->step_plan.k_max, seq, &c->prefill_plan);
    int rc = upload_plan(&c->prefill_plan, c->b.plan_prefill, c->stream);
    if (rc) return rc;
    CU_TRY(cudaMemcpyAsync(c->b.query_tokens, tokens + done, cnt * 4, cudaMemcpyHostToDevice, c->stream));
    rc = run_block(c, kv, c->prefill_plan, nullptr, last);
    if (rc) return rc;
    if ((rc = launch(c->stream, c->pdl, dim3(1), dim3(32), 0, 1, k_prefill_finish, c->prefill_plan.dev,
                     c->step_plan.dev, c->b.state, (const int32_t*)c->b.sel_id, c->b.rec, last ? 1 : 0)))
      return rc;
    c->launches++;
    CU_TRY(cudaStreamSynchronize(c->stream));   // the plan region and token buffer are reused by the next chunk
    done += cnt;
  }
  DevRecord* rh = c->rec_host + seq;
  CU_TRY(cudaMemcpyAsync(rh, c->b.rec + seq, sizeof(DevRecord), cudaMemcpyDeviceToHost, c->stream));
  CU_TRY(cudaStreamSynchronize(c->stream));
  c->len_upper[seq] = rh->new_len;
  c->prefilled[seq] = 1;
  if (out) fill_out(rh, out);
  return rh->status ? BITA_ERR_TIMEOUT : BITA_OK;
}

int bita_prefill(bita_ctx* c, bita_kv* kv, const int32_t* tokens, int32_t count, bita_step_out* out) {
  return bita_prefill_seq(c, kv, 0, tokens, count, out);
}

int bita_step_batch_enqueue(bita_ctx* c, bita_kv* kv, const int32_t* tree_tokens_dev) {
  if (!c || !kv || !kv->k || !kv->v) return BITA_ERR_INVALID_ARG;
  if (kv->C_max != c->m.C_max) return BITA_ERR_INVALID_ARG;
  for (int b = 0; b < c->B; ++b) {
    if (!c->prefilled[b]) return BITA_ERR_NOT_PREFILLED;
    if ((long)c->len_upper[b] + c->step_plan.M > kv->C_max) return BITA_ERR_KV_FULL;
  }
  c->launches = 0;
  int rc = run_block(c, kv, c->step_plan, tree_tokens_dev, true);
  if (rc) return rc;
  if ((rc = launch(c->stream, c->pdl, dim3(c->B), dim3(32), 0, 1, k_accept, c->step_plan.dev, c->b.state,
                   (const int32_t*)c->b.row_token, (const int32_t*)c->b.sel_id, c->b.rec)))
    return rc;
  if ((rc = launch(c->stream, c->pdl, dim3(c->m.L * c->m.H_kv, c->B), dim3(64), 0, 1, k_compact,
                   (const DevRecord*)c->b.rec, c->m.D, kv->C_max, c->m.H_kv, c->B, (bf16*)kv->k, (bf16*)kv->v)))
    return rc;
  c->launches += 2;
  CU_TRY(cudaGetLastError());
  CU_TRY(cudaMemcpyAsync(c->rec_host, c->b.rec, sizeof(DevRecord) * c->B, cudaMemcpyDeviceToHost, c->stream));
  for (int b = 0; b < c->B; ++b) c->len_upper[b] += c->step_plan.max_depth + 1;
  return BITA_OK;
}

int bita_step_batch_finish(bita_ctx* c, bita_step_out* out) {
  if (!c || !out) return BITA_ERR_INVALID_ARG;
  CU_TRY(cudaStreamSynchronize(c->stream));
  int status = 0;
  for (int b = 0; b < c->B; ++b) {
    c->len_upper[b] = c->rec_host[b].new_len;
    fill_out(c->rec_host + b, out + b);
    if (c->rec_host[b].status) status = c->rec_host[b].status;
  }
  return status ? BITA_ERR_TIMEOUT : BITA_OK;
}

int bita_step_batch(bita_ctx* c, bita_kv* kv, const int32_t* tree_tokens, bita_step_out* out) {
  if (!c || !out) return BITA_ERR_INVALID_ARG;
  const int32_t* dev = nullptr;
  const int n = c->B * c->step_plan.N;
  if (tree_tokens && n > 0) {
    for (int i = 0; i < n; ++i)
      if (tree_tokens[i] < -1 || tree_tokens[i] >= c->m.V) return BITA_ERR_INVALID_ARG;
    for (int b = 0; b < c->B; ++b)
      if (!c->prefilled[b]) return BITA_ERR_NOT_PREFILLED;
    CU_TRY(cudaMemcpyAsync(c->b.tree_in, tree_tokens, (size_t)n * 4, cudaMemcpyHostToDevice, c->stream));
    dev = c->b.tree_in;
  }
  int rc = bita_step_batch_enqueue(c, kv, dev);
  if (rc) return rc;
  return bita_step_batch_finish(c, out);
}

/* The batch-1 calls are the batch calls of a context with one sequence. */
int bita_step_enqueue(bita_ctx* c, bita_kv* kv, const int32_t* tree_tokens_dev) {
  if (c && c->B != 1) return BITA_ERR_INVALID_ARG;
  return bita_step_batch_enqueue(c, kv, tree_tokens_dev);
}
int bita_step_finish(bita_ctx* c, bita_step_out* out) {
  if (c && c->B != 1) return BITA_ERR_INVALID_ARG;
  return bita_step_batch_finish(c, out);
}
int bita_step(bita_ctx* c, bita_kv* kv, const int32_t* tree_tokens, bita_step_out* out) {
  if (c && c->B != 1) return BITA_ERR_INVALID_ARG;
  return bita_step_batch(c, kv, tree_tokens, out);
}

int bita_set_debug_buffer(bita_ctx* c, void* dev_buf, size_t bytes) {
  if (!c) return BITA_ERR_INVALID_ARG;
  if (dev_buf) {
    const size_t need = ((size_t)c->m.L * BITA_MAX_ROWS * c->m.d + (size_t)BITA_MAX_ROWS * c->m.V) * 4;
    if (bytes < need) return BITA_ERR_WORKSPACE;
  }
  c->dbg = (float*)dev_buf;
  return BITA_OK;
}

int bita_debug_fetch(bita_ctx* c, int what, void* dst, size_t bytes) {
  if (!c || !dst) return BITA_ERR_INVALID_ARG;
  const size_t rows = (size_t)c->last_rows;
  const void* src = nullptr;
  size_t need = 0;
  if (what == BITA_DEBUG_TOPK) {
    src = c->b.sel_id;
    need = rows * BITA_MAX_TOPK * 4;
  } else if (what == BITA_DEBUG_LOGITS) {
    if (!c->dbg) return BITA_ERR_INVALID_ARG;
    src = c->dbg + (size_t)c->m.L * BITA_MAX_ROWS * c->m.d;
    need = rows * c->m.V * 4;
  } else if (what >= BITA_DEBUG_HIDDEN && what < BITA_DEBUG_HIDDEN + c->m.L) {
    if (!c->dbg) return BITA_ERR_INVALID_ARG;
    src = c->dbg + (size_t)(what - BITA_DEBUG_HIDDEN) * BITA_MAX_ROWS * c->m.d;
    need = rows * c->m.d * 4;
  } else {
    return BITA_ERR_INVALID_ARG;
  }
  if (rows == 0 || bytes < need) return BITA_ERR_INVALID_ARG;
  CU_TRY(cudaMemcpyAsync(dst, src, need, cudaMemcpyDeviceToHost, c->stream));
  CU_TRY(cudaStreamSynchronize(c->stream));
  return BITA_OK;
}

int bita_set_wait_limit(bita_ctx* c, uint64_t limit_ns) {
  if (!c || limit_ns < 1000 || limit_ns > 10000000000ull) return BITA_ERR_INVALID_ARG;
  c->wait_ns = limit_ns;
  return BITA_OK;
}

int bita_probe_wait_timeout(bita_ctx* c, uint64_t limit_ns) {
  if (!c || limit_ns < 1000 || limit_ns > 1000000000ull) return BITA_ERR_INVALID_ARG;
  k_wait_probe<<<1, 32, 0, c->stream>>>(&c->b.state->status, (unsigned long long)limit_ns);
  CU_TRY(cudaGetLastError());
  int32_t status = 0;
  CU_TRY(cudaMemcpyAsync(&status, &c->b.state->status, 4, cudaMemcpyDeviceToHost, c->stream));
  CU_TRY(cudaStreamSynchronize(c->stream));
  return status;
}

int bita_set_kernel_timing(bita_ctx* c, int on) {
  if (!c) return BITA_ERR_INVALID_ARG;
  c->timing = on != 0;
  c->ev_family.clear();
  return BITA_OK;
}

int bita_get_kernel_timing(bita_ctx* c, float* ms, int32_t* launches) {
  if (!c || !ms || !launches) return BITA_ERR_INVALID_ARG;
  CU_TRY(cudaStreamSynchronize(c->stream));
  for (int f = 0; f < BITA_TIMING_FAMILIES; ++f) { ms[f] = 0.f; launches[f] = 0; }
  for (size_t i = 0; i + 1 < c->ev_family.size(); ++i) {
    const int f = c->ev_family[i];
    if (f < 0 || f >= BITA_TIMING_FAMILIES) continue;
    float t = 0.f;
    CU_TRY(cudaEventElapsedTime(&t, c->ev[i], c->ev[i + 1]));
    ms[f] += t;
    launches[f] += c->ev_count[i];
  }
  return BITA_OK;
}

int bita_block_rows(const bita_ctx* c) { return c ? c->step_plan.M : BITA_ERR_INVALID_ARG; }
int bita_last_launch_count(const bita_ctx* c) { return c ? c->launches : BITA_ERR_INVALID_ARG; }

void bita_destroy(bita_ctx* c) {
  if (!c) return;
  cudaStreamSynchronize(c->stream);
  if (c->rec_host) cudaFreeHost(c->rec_host);
  for (cudaEvent_t e : c->ev) cudaEventDestroy(e);
  delete c;
}

const char* bita_strerror(int code) {
  switch (code) {
    case BITA_OK: return "ok";
    case BITA_ERR_INVALID_ARG: return "invalid argument";
    case BITA_ERR_BAD_TEMPLATE: return "bad tree template";
    case BITA_ERR_KV_FULL: return "KV cache full";
    case BITA_ERR_WORKSPACE: return "workspace too small or misaligned";
    case BITA_ERR_CUDA: return "CUDA runtime error";
    case BITA_ERR_TIMEOUT: return "device-side wait timed out";
    case BITA_ERR_NOT_PREFILLED: return "bita_prefill has not been called";
    case BITA_ERR_STATIC_SCRATCH: return "problem exceeds the built-in scratch of the no-allocation entry point";
    default: return "unknown error";
  }
}

int bita_last_cuda_error(void) { return g_last_cuda_error; }

// Workspace of the stand-alone projection: status word, tile counters, split-K exchange buffer.
int bita_gemm_workspace_bytes(int32_t M, int32_t N, int32_t K, size_t* out_bytes) {
  if (!out_bytes || M < 1 || M > BITA_MAX_ROWS || N < 1 || K < 8 || K % 8) return BITA_ERR_INVALID_ARG;
  GemmDesc g;                                                  // shape only: the plan needs no tensor maps
  g.N = N; g.K = K; g.max_splits = 8;
  g.tiles = (N + TC_BLOCK_N - 1) / TC_BLOCK_N;
  g.splits = gemm_splits(g.tiles, K, 8);
  const GemmPlan pl = plan_gemm(g, pad16(M), M);
  const size_t part_tiles = (size_t)pl.tiles * (pl.wide ? 2 : 1) * pl.splits;       // partial tiles of 128 features
  *out_bytes = ALIGN + align_up((size_t)g.tiles * 4) + align_up(pl.splits > 1 ? part_tiles * M * TC_BLOCK_N * 4 : 0);
  return BITA_OK;
}

int bita_gemm_bf16(const void* X, const void* W, void* Y, int32_t M, int32_t N, int32_t K, void* workspace,
                   size_t workspace_bytes, void* cuda_stream) {
  size_t need = 0;
  int rc = bita_gemm_workspace_bytes(M, N, K, &need);
  if (rc) return rc;
  if (!X || !W || !Y) return BITA_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < need || ((uintptr_t)workspace % ALIGN)) return BITA_ERR_WORKSPACE;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  GemmDesc g;
  if ((rc = make_gemm_desc(&g, W, nullptr, N, K, 8))) return rc;
  const int n_pad = pad16(M);
  CUtensorMap mb;
  if ((rc = make_map(&mb, X, K, M, n_pad > 256 ? n_pad / 2 : n_pad))) return rc;
  const size_t cnt_bytes = align_up((size_t)g.tiles * 4);
  CU_TRY(cudaMemsetAsync(workspace, 0, ALIGN + cnt_bytes, s));     // status word and tile counters start at zero
  GemmTcParams p = epi_store((float*)Y, N);
  p.status = (int32_t*)workspace;
  p.tile_counters = (int32_t*)((uint8_t*)workspace + ALIGN);
  p.part = (float*)((uint8_t*)workspace + ALIGN + cnt_bytes);
  p.arrive_target = effective_splits(g, n_pad, M);                 // the counters were just cleared
  if ((rc = launch_gemm_tc(g, mb, n_pad, M, p, false, s))) return rc;
  CU_TRY(cudaGetLastError());
  return BITA_OK;
}

namespace {
size_t attn_partial_bytes(size_t B, size_t H, size_t S, size_t M, size_t D, size_t* acc_offset) {
  const size_t ml = align_up(B * H * S * M * 2 * 4);
  if (acc_offset) *acc_offset = ml;
  return S <= 1 ? 0 : ml + align_up(B * H * S * M * D * 4);
}
}  // namespace

int bita_attention_workspace_bytes_long(int32_t B, int32_t M, int32_t H, int32_t D, int32_t C_max, size_t* out_bytes) {
  size_t base = 0;
  int rc = bita_attention_workspace_bytes(B, M, H, D, &base);
  if (rc) return rc;
  if (C_max < M) return BITA_ERR_INVALID_ARG;
  const int s = attn_balanced_slices(H, B, M, D, C_max);
  const size_t wide = s > 1 ? attn_partial_bytes(B, H, s, M, D, nullptr) : 0;
  *out_bytes = wide > base ? wide : base;
  return BITA_OK;
}

int bita_attention_workspace_bytes(int32_t B, int32_t M, int32_t H, int32_t D, size_t* out_bytes) {
  if (!out_bytes || B < 1 || M < 1 || M > BITA_MAX_ROWS || H < 1 || (D != 64 && D != 128)) return BITA_ERR_INVALID_ARG;
  const size_t S = attn_splits(H, B, M);
  // a single key slice writes its output itself and needs no scratch at all
  *out_bytes = S == 1 ? 0 : align_up((size_t)B * H * S * M * 2 * 4) + align_up((size_t)B * H * S * M * D * 4);
  return BITA_OK;
}

namespace {
int tree_attention_impl(const void* q, const void* k, const void* v, const uint32_t* vis, const void* prompt_k,
                        const void* prompt_v, const uint8_t* sees_prompt, const int32_t* ctx_len, void* out, int32_t B,
                        int32_t M, int32_t H, int32_t H_kv, int32_t D, int32_t P, int32_t C_max, void* workspace,
                        size_t workspace_bytes, void* cuda_stream, int route) {
  size_t need = 0;
  int rc = bita_attention_workspace_bytes(B, M, H, D, &need);
  if (rc) return rc;
  if (!q || !k || !v || !vis || !ctx_len || !out || H_kv < 1 || H % H_kv || P < 0 || P > 64 || C_max < M)
    return BITA_ERR_INVALID_ARG;
  if (P > 0 && (!prompt_k || !prompt_v || !sees_prompt)) return BITA_ERR_INVALID_ARG;
  if (need > 0 && (!workspace || workspace_bytes < need || ((uintptr_t)workspace % ALIGN))) return BITA_ERR_WORKSPACE;
  AttnArgs a{};
  const int W = (M + 31) / 32;
  a.q = (const bf16*)q; a.k = (const bf16*)k; a.v = (const bf16*)v; a.vis = vis;
  a.prompt_k = (const bf16*)prompt_k; a.prompt_v = (const bf16*)prompt_v; a.sees_prompt = sees_prompt;
  a.ctx_len = ctx_len; a.ctx_len_stride = 1; a.vis_batch_stride = M * W; a.sp_batch_stride = M; a.out = (bf16*)out;
  // workspace: partial results of the key slices (used when the slices do not merge inside a cluster).
  // A long cache with a workspace of bita_attention_workspace_bytes_long takes the slice count that
  // makes the waves of CTAs come out even.
  int ws_slices = 0;
  if (route < 0 && g_attention_route == ATTN_ROUTE_AUTO && workspace && !((uintptr_t)workspace % ALIGN)) {
    const int s = attn_balanced_slices(H, B, M, D, C_max);
    if (s > 0 && workspace_bytes >= attn_partial_bytes(B, H, s, M, D, nullptr)) ws_slices = s;
  }
  const size_t S_used = ws_slices > 0 ? (size_t)ws_slices : (size_t)attn_splits(H, B, M);
  size_t acc_off = 0;
  attn_partial_bytes(B, H, S_used, M, D, &acc_off);
  a.part_ml = (float*)workspace;
  a.part_acc = (float*)((uint8_t*)a.part_ml + acc_off);
  a.B = B; a.M = M; a.W = W; a.H = H; a.H_kv = H_kv; a.D = D; a.P = P; a.C_max = C_max;
  if ((rc = launch_attention(a, false, (cudaStream_t)cuda_stream, nullptr, nullptr, route, ws_slices))) return rc;
  CU_TRY(cudaGetLastError());
  return BITA_OK;
}
}  // namespace

int bita_tree_attention(const void* q, const void* k, const void* v, const uint32_t* vis, const void* prompt_k,
                        const void* prompt_v, const uint8_t* sees_prompt, const int32_t* ctx_len, void* out, int32_t B,
                        int32_t M, int32_t H, int32_t H_kv, int32_t D, int32_t P, int32_t C_max, void* workspace,
                        size_t workspace_bytes, void* cuda_stream) {
  return tree_attention_impl(q, k, v, vis, prompt_k, prompt_v, sees_prompt, ctx_len, out, B, M, H, H_kv, D, P, C_max,
                             workspace, workspace_bytes, cuda_stream, -1);
}

int bita_set_attention_route(int route) {
  if (route != ATTN_ROUTE_AUTO && route != ATTN_ROUTE_WORKSPACE) return BITA_ERR_INVALID_ARG;
  g_attention_route = route;
  return BITA_OK;
}

// ---------------------------------------------------------------------------------------------
// No-allocation variant of the tree attention.  Its split-KV partials live in this fixed array of
// the device image instead of caller-provided workspace.  Host code may not hand `g_static_scratch`
// to a kernel (on the host the name is only a handle for the symbol): the device address is
// looked up once per device with cudaGetSymbolAddress and cached.
static __device__ __align__(256) unsigned char g_static_scratch[BITA_STATIC_SCRATCH_BYTES];

namespace {
// Device address of the scratch array on the current device (looked up on first use).
int static_scratch_address(void** out) {
  DeviceFacts* f = device_facts();
  if (!f->static_scratch) {
    void* p = nullptr;
    CU_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
    if (!p || ((uintptr_t)p % ALIGN)) return BITA_ERR_CUDA;
    f->static_scratch = p;
  }
  *out = f->static_scratch;
  return BITA_OK;
}
}  // namespace

int bita_tree_attention_static(const void* q, const void* k, const void* v, const uint32_t* vis, const void* prompt_k,
                               const void* prompt_v, const uint8_t* sees_prompt, const int32_t* ctx_len, void* out,
                               int32_t B, int32_t M, int32_t H, int32_t H_kv, int32_t D, int32_t P, int32_t C_max,
                               void* cuda_stream) {
  size_t need = 0;
  int rc = bita_attention_workspace_bytes(B, M, H, D, &need);
  if (rc) return rc;
  if (need > BITA_STATIC_SCRATCH_BYTES) return BITA_ERR_STATIC_SCRATCH;
  void* scratch = nullptr;
  if (need > 0) {
    rc = static_scratch_address(&scratch);
    if (rc) return rc;
  }
  // The key slices always leave their partial results in the built-in array and the merge kernel
  // reads them back (the workspace route).  Every slot the merge reads was written by the slices
  // of the same call, so nothing in the shared array has to be cleared first.
  return tree_attention_impl(q, k, v, vis, prompt_k, prompt_v, sees_prompt, ctx_len, out, B, M, H, H_kv, D, P, C_max,
                             scratch, need, cuda_stream, ATTN_ROUTE_WORKSPACE);
}

}  // extern "C"
