// Shared device/host declarations of the BiTA step library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bita.h"

#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ < 1000)
#error "this library is written for sm_100a only"
#endif

namespace bita {

typedef __nv_bfloat16 bf16;

// Row kinds of a packed block.
enum RowKind : int32_t { ROW_ROOT = 0, ROW_NODE = 1, ROW_MASK = 2, ROW_QUERY = 3 };

// Layout of one packed block as the kernels see it (all pointers DEVICE).  A block holds the rows
// of B sequences, sequence-major: global row b * M + r is row r of the block's b-th sequence, which
// is sequence seq0 + b of the context.  Every table below describes ONE sequence's M rows.
struct DevPlan {
  int32_t M;                  // rows per sequence
  int32_t B;                  // sequences in the block
  int32_t seq0;               // first of them
  int32_t W;                  // 32-bit words per visibility row = ceil(M / 32)
  int32_t N;                  // tree nodes
  int32_t G;                  // mask groups
  int32_t n_mask;
  int32_t k_max;              // top-k width kept per mask row
  int32_t n_query;            // prefill: query tokens in this chunk (rows 0..n_query-1), else 0
  int32_t max_depth;
  const int32_t* row_kind;    // [M]
  const int32_t* row_idx;     // [M] node index / mask index within its group / query index
  const int32_t* rel_pos;     // [M] position id minus C
  const uint8_t* sees_prompt; // [M]
  const uint32_t* vis;        // [M][W]
  const int32_t* parent;      // [N]
  const int32_t* rank;        // [N]
  const int32_t* depth;       // [N]
  const int32_t* group_of;    // [N + 1] group attached to node i-1 (index 0 = root), or -1
};

// Decoding state that lives on the device between passes.
struct DevState {
  int32_t len;                // C: tokens in the cache
  int32_t root;               // last accepted token
  int32_t status;             // sticky error word (0 = fine)
  int32_t pad;
  int32_t tree[BITA_MAX_NODES];
};

// Device-side result record (mirrors bita_step_out, plus what compaction needs).
struct DevRecord {
  int32_t status;
  int32_t n_out;
  int32_t new_len;
  int32_t out_tokens[BITA_MAX_DEPTH + 1];
  int32_t accepted_idx[BITA_MAX_DEPTH];
  int32_t next_tree[BITA_MAX_NODES];
  int32_t old_len;            // C before the pass
  int32_t n_acc;              // accepted drafts
};

__device__ __forceinline__ float bf2f(bf16 v) { return __bfloat162float(v); }
__device__ __forceinline__ bf16 f2bf(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Programmatic dependent launch: `pdl_launch` lets the next kernel of the stream begin its own
// prologue; `pdl_wait` blocks until every kernel this one depends on has completed and its writes
// are visible.  A kernel must not touch memory that earlier kernels write before `pdl_wait`.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
}  // namespace bita
