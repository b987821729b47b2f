// Internal declarations shared by the library's translation units.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "aspd.h"

namespace aspd {

constexpr int kMaxRowsPerItem = 64;   // query rows (tokens x group heads) one work item carries
constexpr int kCausalAll = 1 << 29;   // causal0 value of a fully visible chunk

// ---------------------------------------------------------------------------------------
// Cache tile format.  One (page, KV head) tile holds page_size tokens x head_dim elements.
// A token row is cut into 128-byte spans; span s of all tokens is stored together as
// [page_size][128 B], and inside it the 16-byte chunk index is XOR-ed with (token & 7).
// That is the 128-byte-swizzled, K-major shared-memory image the tensor-core and ldmatrix
// paths want, so a tile lands in shared memory with linear bulk copies and no re-layout.
// ---------------------------------------------------------------------------------------
__host__ __device__ inline size_t tile_bytes(int page_size, int head_dim, int esize) {
  return (size_t)page_size * head_dim * esize;
}
// Byte offset, inside a tile, of byte `b` (multiple of the element size) of token `t`'s row.
__host__ __device__ inline uint32_t tile_offset(int t, uint32_t b, int page_size) {
  uint32_t span = b >> 7, in = b & 127u;
  return span * (uint32_t)page_size * 128u + (uint32_t)t * 128u + ((((in >> 4) ^ (uint32_t)(t & 7)) << 4) | (in & 15u));
}

struct DeviceItem {       // mirrors aspd_item_t, 32 bytes
  int32_t q_tok0, n_q_tok, kv_head, page0, n_keys, causal0, part_slot, request;
};

struct PlanDevice {       // pointers into the plan's single device allocation
  const DeviceItem* items;
  const int32_t* page_ids;     // concatenated page tables (physical page per logical page)
  const int32_t* tok_page;     // [n_new] physical page the new token's K/V goes to
  const int32_t* tok_row;      // [n_new] row inside that page
  const float2* q_cs;          // [n_new][head_dim/2] (cos, sin) of the query's RoPE angle
  const int32_t* part_base;    // [n_new + 1] first partial record of each new token
  const double* inv_freq;      // [head_dim/2]
  float* ws_o;                 // [n_partials][n_q_heads][head_dim] un-normalised partial outputs
  float2* ws_ml;               // [n_partials][n_q_heads] (running max in log2 units, sum)
  int32_t* status;             // first error recorded by a kernel
  int32_t* work_counter;       // dynamic work-list cursor (reset by its last reader)
  // staging for aspd_step_host
  void* st_q; void* st_k; void* st_v; void* st_out; int32_t* st_pos;
};

}  // namespace aspd

struct aspd_plan {
  aspd_shape_t shape;
  int mode;
  int n_req;
  int n_new;
  int n_items;
  int n_partials;
  int kernel;
  int chunk_tokens;
  int n_ctas;
  int host_only;
  int sm_count;
  int64_t n_pool_pages;
  int64_t kv_tokens_read;
  int64_t algorithmic_bytes;
  size_t device_bytes;
  void* device_base;
  aspd::PlanDevice dev;
  std::vector<aspd::DeviceItem> items;
};

namespace aspd {
// launchers (each returns an aspd_status_t)
int launch_append(const aspd_plan* p, const void* k_new, const void* v_new, const int32_t* pos,
                  void* k_pool, void* v_pool, cudaStream_t s);
int launch_attn_generic(const aspd_plan* p, const void* q, const void* k_pool, const void* v_pool,
                        cudaStream_t s);
int launch_attn_mma(const aspd_plan* p, const void* q, const void* k_pool, const void* v_pool,
                    cudaStream_t s);
int launch_combine(const aspd_plan* p, void* out, cudaStream_t s);
int launch_read_token(const aspd_shape_t* shape, const void* pool, int64_t page, int row, int kv_head,
                      float* out_dev, cudaStream_t s);
inline int esize_of(int dtype) { return dtype == ASPD_DTYPE_BF16 ? 2 : 4; }
}  // namespace aspd
