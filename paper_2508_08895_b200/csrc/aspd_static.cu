// aspd_attn_static: the attention of a step with every byte of scratch in a device array that
// is part of the library image, for callers that cannot allocate device memory.
#include <math.h>
#include <string.h>

#include <mutex>
#include <vector>

#include "aspd_internal.cuh"

using namespace aspd;

namespace {

// The scratch.  In host code `g_scratch` is only a handle for the symbol, not a device address;
// the address a kernel may use comes from cudaGetSymbolAddress (below).
static __device__ __align__(256) unsigned char g_scratch[ASPD_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mu;      // two host threads making their first call on a device at the same time

// Device address of the scratch array on the current device (looked up once per device).
int scratch_address(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ASPD_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mu);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_scratch) != cudaSuccess || !ptr) return ASPD_ERR_CUDA;
    g_scratch_addr[dev] = static_cast<unsigned char*>(ptr);
  }
  *out = g_scratch_addr[dev];
  return ASPD_OK;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// The status word sits at a fixed place, the array's last 256 bytes, so that aspd_static_status
// finds it whatever the last call's tables looked like.
constexpr size_t kStatusOffset = ASPD_STATIC_SCRATCH_BYTES - 256;

}  // namespace

extern "C" int aspd_attn_static(const aspd_plan_t* plan, const void* q, const void* k_pool, const void* v_pool, void* out,
                                void* stream) {
  if (!plan || !plan->host_only) return ASPD_ERR_INVALID_ARG;
  if (plan->n_new == 0) return ASPD_OK;
  if (!q || !k_pool || !v_pool || !out || aspd::misaligned16(q, k_pool, v_pool, out)) return ASPD_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  // The tables go up from pageable memory of this call: such a copy cannot be recorded into a
  // graph (a replay would read a buffer that is gone), so a capturing stream is refused.
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &capturing) != cudaSuccess) return ASPD_ERR_CUDA;
  if (capturing != cudaStreamCaptureStatusNone) return ASPD_ERR_UNSUPPORTED;
  const aspd_shape_t& sh = plan->shape;
  const int d = sh.head_dim, G = sh.n_q_heads / sh.n_kv_heads, n_new = plan->n_new;

  // layout of the tables and of the split-K workspace inside the scratch array
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t o_items = take(sizeof(DeviceItem) * plan->items.size());
  const size_t o_cta = take(sizeof(int4) * (size_t)(plan->n_ctas > 0 ? plan->n_ctas : 1));
  const size_t o_visit = take(sizeof(int2) * plan->visit.size());
  const size_t o_tvis = take(sizeof(int4) * plan->tok_vis.size());
  const size_t o_rb = take(sizeof(int2) * plan->row_blocks.size());
  const size_t o_qcs = take(sizeof(float2) * (size_t)n_new * (d / 2));
  const size_t o_pbase = take(sizeof(int32_t) * plan->part_base.size());
  const size_t upload_bytes = off;
  const size_t o_wso = take(sizeof(float) * (size_t)plan->n_partials * G * d);
  const size_t o_wsml = take(sizeof(float2) * (size_t)plan->n_partials * G);
  if (off > kStatusOffset) return ASPD_ERR_TOO_LARGE;

  unsigned char* base = nullptr;
  int rc = scratch_address(&base);
  if (rc) return rc;

  // tables: everything that must start from a known value is rewritten here (the status word
  // and the work counter start at zero; the workspace is fully written before it is read)
  std::vector<uint8_t> blob(upload_bytes, 0);
  memcpy(blob.data() + o_items, plan->items.data(), sizeof(DeviceItem) * plan->items.size());
  aspd::fill_cta_head(plan, reinterpret_cast<int4*>(blob.data() + o_cta));
  memcpy(blob.data() + o_visit, plan->visit.data(), sizeof(int2) * plan->visit.size());
  memcpy(blob.data() + o_tvis, plan->tok_vis.data(), sizeof(int4) * plan->tok_vis.size());
  memcpy(blob.data() + o_rb, plan->row_blocks.data(), sizeof(int2) * plan->row_blocks.size());
  memcpy(blob.data() + o_pbase, plan->part_base.data(), sizeof(int32_t) * plan->part_base.size());
  float2* qcs = reinterpret_cast<float2*>(blob.data() + o_qcs);
  double inv_freq[64];
  for (int i = 0; i < d / 2; ++i) inv_freq[i] = pow((double)sh.rope_theta, -2.0 * i / d);
  for (int t = 0; t < n_new; ++t)
    for (int i = 0; i < d / 2; ++i) {
      const double a = (double)plan->q_pos[t] * inv_freq[i];
      qcs[(size_t)t * (d / 2) + i] = make_float2((float)cos(a), (float)sin(a));
    }
  // the source is pageable host memory: the copy is staged before the call returns (the host may
  // wait for earlier work on the stream); the status word and the work counter start at zero
  if (cudaMemcpyAsync(base, blob.data(), upload_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemsetAsync(base + kStatusOffset, 0, 2 * sizeof(int32_t), s) != cudaSuccess)
    return ASPD_ERR_CUDA;

  // a shell of the plan whose device pointers all lie inside the scratch array
  aspd_plan shell;
  shell.shape = plan->shape; shell.mode = plan->mode; shell.n_req = plan->n_req; shell.n_new = plan->n_new;
  shell.n_items = plan->n_items; shell.n_partials = plan->n_partials; shell.kernel = plan->kernel;
  shell.chunk_tokens = plan->chunk_tokens; shell.n_ctas = plan->n_ctas; shell.host_only = 0;
  shell.sm_count = plan->sm_count; shell.n_row_blocks = plan->n_row_blocks; shell.stable_cache = 0; shell.fuse_append = 0; shell.n_pool_pages = plan->n_pool_pages;
  shell.kv_tokens_read = plan->kv_tokens_read; shell.algorithmic_bytes = plan->algorithmic_bytes;
  shell.dealt = plan->dealt; shell.wide = plan->wide; shell.shared_mask = plan->shared_mask; shell.m64 = plan->m64;   // which kernel variant the items were made for
  shell.device_bytes = 0; shell.device_base = nullptr;
  memset(&shell.dev, 0, sizeof(shell.dev));
  shell.dev.items = (const DeviceItem*)(base + o_items);
  shell.dev.cta_head = (const int4*)(base + o_cta);
  shell.dev.visit = (const int2*)(base + o_visit);
  shell.dev.tok_vis = (const int4*)(base + o_tvis);
  shell.dev.row_blocks = (const int2*)(base + o_rb);
  shell.dev.q_cs = (const float2*)(base + o_qcs);
  shell.dev.part_base = (const int32_t*)(base + o_pbase);
  shell.dev.status = (int32_t*)(base + kStatusOffset);
  shell.dev.work_counter = shell.dev.status + 1;
  shell.dev.ws_o = (float*)(base + o_wso);
  shell.dev.ws_ml = (float2*)(base + o_wsml);
  shell.dev.pool_limit = (int32_t)plan->n_pool_pages;

  // plans that deal whole streams have one item per (token, KV head): their kernel writes the output
  if (attn_mma_direct(&shell)) return launch_attn_mma(&shell, q, k_pool, v_pool, out, s);
  rc = shell.kernel == ASPD_KERNEL_MMA ? launch_attn_mma(&shell, q, k_pool, v_pool, nullptr, s)
                                       : launch_attn_generic(&shell, q, k_pool, v_pool, s);
  if (rc) return rc;
  return launch_combine(&shell, out, s);
}

extern "C" int aspd_static_status(void* stream) {
  unsigned char* base = nullptr;
  int rc = scratch_address(&base);
  if (rc) return rc;
  int32_t st = 0;
  cudaStream_t s = (cudaStream_t)stream;
  if (cudaMemcpyAsync(&st, base + kStatusOffset, sizeof(st), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return ASPD_ERR_CUDA;
  return st;
}
