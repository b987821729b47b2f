// Internal declarations shared by the library's translation units.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "aspd.h"

namespace aspd {

constexpr int kMaxRowsPerItem = 64;   // query rows (tokens x group heads) one work item carries
constexpr int kMaxRowsWide = 128;     // ... in a plan that deals whole streams to the tensor-core kernel's CTAs
constexpr int kCausalAll = 1 << 29;   // prefix end of a token that sees its whole key stream

// ---------------------------------------------------------------------------------------
// Cache tile format.  One (page, KV head) tile holds page_size tokens x head_dim elements,
// row_bytes = head_dim * element size per token.  Tokens are taken in groups of 8 and a token
// row is cut into 128-byte spans; the tile is stored as [token group][span][8 tokens][128 B],
// and inside each 1 KiB block the 16-byte chunk index is XOR-ed with (token & 7).  Every 1 KiB
// block is a 128-byte-swizzle atom of the tensor core's shared-memory operands, and the blocks
// of one span lie a constant 8 * row_bytes apart even across consecutive tiles, so whole tiles
// copied back to back into shared memory (one linear bulk copy each) form a valid K-major
// operand (keys x head_dim, for Q.K^T) and MN-major operand (head_dim x keys, for P.V) as is.
// ---------------------------------------------------------------------------------------
__host__ __device__ inline size_t tile_bytes(int page_size, int head_dim, int esize) {
  return (size_t)page_size * head_dim * esize;
}
// Byte offset, inside a tile, of byte `b` (multiple of the element size) of token `t`'s row.
__host__ __device__ inline uint32_t tile_offset(int t, uint32_t b, uint32_t row_bytes) {
  const uint32_t span = b >> 7, in = b & 127u;
  return (uint32_t)(t >> 3) * (8u * row_bytes) + span * 1024u + (uint32_t)(t & 7) * 128u +
         ((((in >> 4) ^ (uint32_t)(t & 7)) << 4) | (in & 15u));
}

struct DeviceItem {       // mirrors aspd_item_t, 40 bytes
  int32_t q_tok0, n_q_tok, kv_head, page0, n_pages, key0, part_slot, request, row_block, n_parts;   // n_parts: items its stream was cut into
};

struct PlanDevice {       // pointers into the plan's single device allocation
  const DeviceItem* items;
  const int4* cta_head;        // [n_ctas] (first item, end item, page0 and n_pages of the first item): everything a CTA
                               // needs to request its first pages comes with one load
  const int2* visit;           // key streams, per page to read: (physical page, valid rows | new rows << 8 |
                               // first new token << 13); the new rows are the last valid rows of the page
  const int32_t* cta_dirty0;   // [n_ctas + 1] range of `dirty` that CTA c must write before reading (fused step)
  const int4* dirty;           // (physical page, KV head, new token, row) of every new row in a CTA's pages
  const int4* tok_vis;         // [n_new] (pe, lo, hi, -): visible stream keys are [0, pe) and [lo, hi)
  const int2* row_blocks;      // [n_row_blocks] (first new token, number of tokens)
  const int32_t* tok_page;     // [n_new] physical page the new token's K/V goes to
  const int32_t* tok_row;      // [n_new] row inside that page
  const int32_t* tok_pos;      // [n_new] position ID of the new token as the plan derived it (or q_pos)
  const float2* q_cs;          // [n_new][head_dim/2] (cos, sin) of the query's RoPE angle
  const int32_t* part_base;    // [n_new * n_kv_heads + 1] first partial record of (new token, KV head)
  const double* inv_freq;      // [head_dim/2]
  float* ws_o;                 // [n_partials][G][head_dim] un-normalised partial outputs
  float2* ws_ml;               // [n_partials][G] (reference max in log2 units, sum)
  int32_t* status;             // first error recorded by a kernel
  int32_t* work_counter;       // dynamic work-list cursor (reset by its last reader)
  int32_t* arrive;             // [n_new * n_kv_heads] records of (new token, KV head) stored so far in this launch (plans
                               // that merge inside the attention kernel; zero between launches)
  // staging for aspd_step_host
  void* st_q; void* st_k; void* st_v; void* st_out; int32_t* st_pos;
  int32_t pool_limit;          // pages in each pool: what builds with -DASPD_DEBUG_BOUNDS check page ids against
};

// Builds with -DASPD_DEBUG_BOUNDS: a kernel that meets a page id or row outside the pool records
// ASPD_ERR_BAD_DESCRIPTOR in the plan's status word and leaves the access out (nothing traps).
// Host validation makes this unreachable for plans the library built; the check is there for the
// development of the planner and of the kernels' index arithmetic.
#ifdef ASPD_DEBUG_BOUNDS
__device__ __forceinline__ bool bounds_ok(const PlanDevice& pd, int page, int row, int page_size) {
  if (page >= 0 && page < pd.pool_limit && row >= 0 && row < page_size) return true;
  atomicCAS(pd.status, 0, (int)ASPD_ERR_BAD_DESCRIPTOR);
  return false;
}
#else
__device__ __forceinline__ bool bounds_ok(const PlanDevice&, int, int, int) { return true; }
#endif

}  // namespace aspd

namespace aspd {
// Byte offsets of the plan's tables inside its device block, and how many entries the
// length-dependent ones have room for.
struct PlanLayout {
  size_t o_items = 0, o_cta = 0, o_visit = 0, o_cdirty = 0, o_dirty = 0, o_tpage = 0, o_trow = 0, o_tpos = 0, o_tvis = 0,
         o_rb = 0, o_pbase = 0, o_freq = 0, o_status = 0, o_arrive = 0, upload_bytes = 0, o_qcs = 0, o_wso = 0, o_wsml = 0, o_stq = 0,
         o_stk = 0, o_stv = 0, o_sto = 0, o_stp = 0, device_bytes = 0;
  size_t cap_items = 0, cap_visit = 0, cap_dirty = 0, cap_partials = 0, n_row_blocks = 0, n_part_base = 0;
};
}  // namespace aspd

struct aspd_plan {
  aspd_shape_t shape = {};
  int mode = 0;
  int n_req = 0;
  int n_new = 0;
  int n_items = 0;
  int n_partials = 0;
  int kernel = 0;
  int chunk_tokens = 0;
  int n_ctas = 0;
  int host_only = 0;
  int sm_count = 0;
  int n_row_blocks = 0;
  int fuse_append = 0;             // few enough new rows per CTA for the attention pass to write them itself
  int stable_cache = 0;            // producers may fetch pages without new rows before the dependency wait
  int dealt = 0;                   // whole streams dealt to the CTAs in turn (many more streams than CTAs)
  int shared_mask = 0;             // parallel step under the ablation's visible mask
  int wide = 0;                    // dealt plan of the tensor-core kernel: row blocks of up to kMaxRowsWide rows
  int m64 = 0;                     // stream-K plan of the tensor-core kernel whose MMAs take M = 64 (row blocks are at most 64 rows)
  int stagger_start = 0;           // few tiles per CTA: order the requests of a CTA's first tiles (see the producers)
  int single_launch = 0;           // stream-K plan of the tensor-core kernel whose last-arriving CTAs merge the records themselves
  int64_t n_pool_pages = 0;
  int64_t kv_tokens_read = 0;
  int64_t algorithmic_bytes = 0;
  size_t device_bytes = 0;
  void* host_block = nullptr;      // page-locked host buffer the tables were assembled in (travels with the device block)
  size_t host_block_bytes = 0;
  cudaEvent_t upload_done = nullptr;   // recorded after the table copy: the host buffer may be rewritten once it has completed
  size_t block_bytes = 0;          // size of the device block the plan holds (a reused block may be larger than needed)
  std::vector<cudaStream_t> streams;   // streams the plan's work was enqueued on
  void* device_base = nullptr;
  aspd::PlanDevice dev = {};
  std::vector<aspd::DeviceItem> items;
  std::vector<int2> visit;
  std::vector<int4> tok_vis;
  // further host copies of the plan's tables (what the device allocation is filled from)
  std::vector<int32_t> cta_item0, part_base, q_pos;
  std::vector<int2> row_blocks;
  std::vector<int32_t> tok_page, tok_row, cta_dirty0;
  std::vector<int4> dirty;
  aspd_tuning_t tune = {};
  aspd::PlanLayout layout;
};

namespace aspd {
// Programmatic dependent launch.  Every kernel of the library is launched with the
// "programmatic stream serialization" attribute and begins with pdl_enter(): it lets the next
// kernel in the stream start its own set-up right away and then waits until the previous kernel
// has completed and its writes are visible.  Because every kernel waits before it ends, the
// dependency on all earlier kernels of the stream is kept transitively; what is gained is that
// launch latency and set-up of a kernel overlap the tail of the one before it.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

enum { kPdlAppend = 1, kPdlAttn = 2, kPdlCombine = 4, kPdlCombineLarge = 8 };
// which kernels are launched with the attribute: append, attention, and the combine of large steps
constexpr int pdl_mask() { return kPdlAppend | kPdlAttn | kPdlCombineLarge; }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(int which, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = (pdl_mask() & which) ? 1 : 0;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// launchers (each returns an aspd_status_t)
int launch_append(const aspd_plan* p, const void* k_new, const void* v_new, const int32_t* pos,
                  void* k_pool, void* v_pool, cudaStream_t s);
int launch_attn_generic(const aspd_plan* p, const void* q, const void* k_pool, const void* v_pool,
                        cudaStream_t s);
// out: null = (m, l, O) records for the combine kernel; non-null = final output, written by the
// kernel itself when the plan has one item per (token, KV head) (ignored otherwise)
int launch_attn_mma(const aspd_plan* p, const void* q, const void* k_pool, const void* v_pool, void* out,
                    cudaStream_t s);
inline bool attn_mma_direct(const aspd_plan* p) { return p->kernel == ASPD_KERNEL_MMA && p->dealt; }   // one item per (token, KV head)
inline bool attn_mma_writes_output(const aspd_plan* p) { return attn_mma_direct(p) || (p->kernel == ASPD_KERNEL_MMA && p->single_launch); }
int launch_combine(const aspd_plan* p, void* out, cudaStream_t s);
// fills the plan's cos/sin table from its position and frequency tables (plan creation, after the upload)
int launch_qcs(const aspd_plan* p, cudaStream_t s);
// attention pass that first writes this step's new K (rotated) and V rows into the pages it reads
int launch_attn_mma_step(const aspd_plan* p, const void* q, const void* k_new, const void* v_new, void* k_pool,
                         void* v_pool, void* out, cudaStream_t s);
int launch_rerotate(const aspd_shape_t* shape, void* k_pool, const int32_t* pages, const int32_t* rows, const int32_t* delta,
                    int n, cudaStream_t s);
int launch_rerotate_ranges(const aspd_shape_t* shape, void* const* k_pools, int n_layers, const int32_t* page_table,
                           const int32_t* ranges, int n_ranges, cudaStream_t s);
int set_profile_buffer(long long* device_buf, int cta);
int launch_wait_probe(long long limit_cycles, int32_t* status_dev, cudaStream_t s);
int launch_read_token(const aspd_shape_t* shape, const void* pool, int64_t page, int row, int kv_head,
                      float* out_dev, cudaStream_t s);
// the per-CTA head table of the device plan, from the host tables
inline void fill_cta_head(const aspd_plan* p, int4* dst) {
  for (int c = 0; c < p->n_ctas; ++c) {
    const int b = p->cta_item0[c], e = p->cta_item0[c + 1];
    dst[c] = make_int4(b, e, b < e ? p->items[b].page0 : 0, b < e ? p->items[b].n_pages : 0);
  }
}
inline int esize_of(int dtype) { return dtype == ASPD_DTYPE_BF16 ? 2 : 4; }
// device buffers are moved in 16-byte pieces: a pointer off that boundary is refused, not dereferenced
inline bool misaligned16(const void* a, const void* b = nullptr, const void* c = nullptr, const void* d = nullptr,
                         const void* e = nullptr, const void* f = nullptr) {
  return ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b) | reinterpret_cast<uintptr_t>(c) |
           reinterpret_cast<uintptr_t>(d) | reinterpret_cast<uintptr_t>(e) | reinterpret_cast<uintptr_t>(f)) & 15u) != 0;
}
}  // namespace aspd
