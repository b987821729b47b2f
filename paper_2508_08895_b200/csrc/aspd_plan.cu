// Host side of the library: descriptor validation, position IDs and slots (integer rules of
// Eq. 4 and Section 3.3), the split-K work list, plan life cycle and the C entry points.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <new>
#include <vector>

#include "aspd_internal.cuh"

using namespace aspd;

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- device blocks of destroyed plans are kept for the next plan --------------------------------
// A decode loop makes a new plan every step; cudaMalloc and cudaFree (which waits for the whole
// device) would cost more than the step's host work.  aspd_plan_destroy therefore parks the plan's
// block together with an event recorded on every stream the plan was used on, and
// aspd_plan_create takes a parked block of fitting size and makes its stream wait for those events
// before the new tables are uploaded -- no host synchronisation on either side.  With the block goes
// the page-locked host buffer the tables are assembled in (a copy from pageable memory would make
// the host wait for everything queued before it on the stream).
// upload_done: recorded right after the plan's table copy; the host may write the buffer again only
// once it has completed, so a block whose copy is still queued is passed over (a fresh one is
// allocated instead and the pool settles at the depth the loop needs).
struct ParkedBlock { void* ptr; size_t bytes; void* host; size_t host_bytes; int device; cudaEvent_t upload_done; std::vector<cudaEvent_t> events; };
std::mutex g_blocks_mu;
std::vector<ParkedBlock> g_blocks;
constexpr size_t kParkedMax = 8;                       // blocks kept per process
constexpr size_t kParkedMaxBytes = 2048ull << 20;     // all parked blocks together; what does not fit is freed right away

int block_acquire(size_t bytes, size_t host_need, cudaStream_t s, void** out, size_t* got, void** host, size_t* host_got) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ASPD_ERR_CUDA;
  {
    std::lock_guard<std::mutex> lock(g_blocks_mu);
    int best = -1, oldest = -1, fitting = 0;
    for (int i = 0; i < (int)g_blocks.size(); ++i) {
      if (g_blocks[i].device != dev || g_blocks[i].bytes < bytes || g_blocks[i].bytes > 4 * bytes + (1u << 20)) continue;
      ++fitting;
      if (oldest < 0) oldest = i;
      if ((best < 0 || g_blocks[i].bytes < g_blocks[best].bytes) &&
          (g_blocks[i].upload_done == nullptr || cudaEventQuery(g_blocks[i].upload_done) == cudaSuccess))
        best = i;
    }
    // every fitting block still has its copy queued: with a couple of them parked the host is simply
    // ahead of the GPU and waits for the oldest one instead of allocating more
    if (best < 0 && fitting >= 2 && cudaEventSynchronize(g_blocks[oldest].upload_done) == cudaSuccess) best = oldest;
    if (best >= 0) {
      ParkedBlock b = g_blocks[best];
      g_blocks.erase(g_blocks.begin() + best);
      int rc = ASPD_OK;
      if (b.upload_done) cudaEventDestroy(b.upload_done);
      for (cudaEvent_t e : b.events) {
        if (cudaStreamWaitEvent(s, e, 0) != cudaSuccess) rc = ASPD_ERR_CUDA;
        cudaEventDestroy(e);
      }
      if (rc == ASPD_OK && b.host_bytes < host_need) {           // too small for the new tables (its last copy has completed)
        cudaFreeHost(b.host);
        b.host = nullptr; b.host_bytes = 0;
        if (rc == ASPD_OK && cudaMallocHost(&b.host, host_need) != cudaSuccess) rc = ASPD_ERR_NOMEM;
        if (rc == ASPD_OK) b.host_bytes = host_need;
      }
      if (rc) { cudaFree(b.ptr); if (b.host) cudaFreeHost(b.host); return rc; }
      *out = b.ptr; *got = b.bytes; *host = b.host; *host_got = b.host_bytes;
      return ASPD_OK;
    }
  }
  if (cudaMalloc(out, bytes) != cudaSuccess) return ASPD_ERR_NOMEM;
  if (cudaMallocHost(host, host_need) != cudaSuccess) { cudaFree(*out); return ASPD_ERR_NOMEM; }
  *got = bytes; *host_got = host_need;
  return ASPD_OK;
}

int block_release(void* ptr, size_t bytes, void* host, size_t host_bytes, cudaEvent_t upload_done,
                  const std::vector<cudaStream_t>& streams) {
  int dev = 0;
  bool park = cudaGetDevice(&dev) == cudaSuccess;
  cudaPointerAttributes attr;
  if (park && (cudaPointerGetAttributes(&attr, ptr) != cudaSuccess || attr.device != dev)) park = false;   // freed from another device's context
  std::vector<cudaEvent_t> events;
  for (size_t i = 0; park && i < streams.size(); ++i) {
    cudaEvent_t e;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { park = false; break; }
    if (cudaEventRecord(e, streams[i]) != cudaSuccess) { cudaEventDestroy(e); park = false; break; }   // e.g. the stream is gone
    events.push_back(e);
  }
  if (park) {
    std::lock_guard<std::mutex> lock(g_blocks_mu);
    size_t parked = 0;
    for (const ParkedBlock& b : g_blocks) parked += b.bytes;
    if (g_blocks.size() < kParkedMax && parked + bytes <= kParkedMaxBytes) {
      g_blocks.push_back({ptr, bytes, host, host_bytes, dev, upload_done, events});
      return ASPD_OK;
    }
  }
  for (cudaEvent_t e : events) cudaEventDestroy(e);
  if (upload_done) cudaEventDestroy(upload_done);
  const bool ok = cudaFree(ptr) == cudaSuccess;      // waits for the device: the buffer's last copy is done after it
  if (host) cudaFreeHost(host);
  return ok ? ASPD_OK : ASPD_ERR_CUDA;
}

int block_cache_clear() {
  std::vector<ParkedBlock> all;
  {
    std::lock_guard<std::mutex> lock(g_blocks_mu);
    all.swap(g_blocks);
  }
  int rc = ASPD_OK;
  for (ParkedBlock& b : all) {
    for (cudaEvent_t e : b.events) cudaEventDestroy(e);
    if (b.upload_done) cudaEventDestroy(b.upload_done);
    if (cudaFree(b.ptr) != cudaSuccess) rc = ASPD_ERR_CUDA;
    if (b.host) cudaFreeHost(b.host);
  }
  return rc;
}

// every stream a plan's work was enqueued on (a handful at most): what its block must wait for when reused
inline void note_stream(aspd_plan* p, void* stream) {
  cudaStream_t s = (cudaStream_t)stream;
  if (std::find(p->streams.begin(), p->streams.end(), s) == p->streams.end()) p->streams.push_back(s);
}

int check_shape(const aspd_shape_t* s) {
  if (!s) return ASPD_ERR_INVALID_ARG;
  if (s->n_q_heads <= 0 || s->n_kv_heads <= 0 || s->n_q_heads % s->n_kv_heads) return ASPD_ERR_INVALID_ARG;
  if (s->head_dim != 64 && s->head_dim != 128) return ASPD_ERR_UNSUPPORTED;
  if (s->dtype != ASPD_DTYPE_F32 && s->dtype != ASPD_DTYPE_BF16) return ASPD_ERR_UNSUPPORTED;
  if (s->page_size != 8 && s->page_size != 16 && s->page_size != 32) return ASPD_ERR_UNSUPPORTED;
  if (s->n_q_heads / s->n_kv_heads > kMaxRowsPerItem) return ASPD_ERR_UNSUPPORTED;
  if (!(s->rope_theta > 0.f) || !(s->sm_scale > 0.f)) return ASPD_ERR_INVALID_ARG;
  return ASPD_OK;
}

// Structural checks that need no page table: counts, q_len <= kv_len, tail in serial mode.
int check_counts(const aspd_request_t* req, const aspd_branch_t* br, int n_req, int mode) {
  if (n_req < 0 || (n_req > 0 && !req)) return ASPD_ERR_INVALID_ARG;
  if (mode != ASPD_MODE_BRANCH && mode != ASPD_MODE_SERIAL) return ASPD_ERR_INVALID_ARG;
  for (int r = 0; r < n_req; ++r) {
    const aspd_request_t& q = req[r];
    if (q.prefix_len < 0 || q.n_branches < 0 || q.branch_begin < 0 || q.tail_len < 0 || q.tail_off < 0)
      return ASPD_ERR_BAD_DESCRIPTOR;
    if (q.n_branches > 0 && !br) return ASPD_ERR_INVALID_ARG;
    for (int b = 0; b < q.n_branches; ++b) {
      const aspd_branch_t& x = br[q.branch_begin + b];
      if (x.kv_off < 0 || x.kv_len < 0 || x.q_len < ASPD_Q_SHARED || x.q_len > x.kv_len || x.pos_start < ASPD_POS_AUTO)
        return ASPD_ERR_BAD_DESCRIPTOR;
    }
    if (mode == ASPD_MODE_SERIAL && q.tail_len < 1) return ASPD_ERR_BAD_DESCRIPTOR;
  }
  return ASPD_OK;
}

struct Region { int lo, hi; };

// Regions inside the page table, page alignment, overlap, page ids.
int check_layout(const aspd_shape_t* s, const aspd_request_t* req, const aspd_branch_t* br, const int32_t* page_ids,
                 int n_req, int64_t n_pool_pages, int mode) {
  if (n_req > 0 && !page_ids) return ASPD_ERR_INVALID_ARG;
  if (n_pool_pages < 0) return ASPD_ERR_INVALID_ARG;
  std::vector<uint8_t> used((size_t)n_pool_pages, 0);
  std::vector<Region> regs;
  for (int r = 0; r < n_req; ++r) {
    const aspd_request_t& q = req[r];
    if (q.page_begin < 0 || q.n_pages < 0) return ASPD_ERR_BAD_DESCRIPTOR;
    const long cap = (long)q.n_pages * s->page_size;
    regs.clear();
    regs.push_back({0, q.prefix_len});
    for (int b = 0; b < q.n_branches; ++b) {
      const aspd_branch_t& x = br[q.branch_begin + b];
      if (x.kv_off % s->page_size) return ASPD_ERR_BAD_DESCRIPTOR;
      regs.push_back({x.kv_off, x.kv_off + x.kv_len});
    }
    if (mode == ASPD_MODE_SERIAL || q.tail_len > 0) {
      if (q.tail_off % s->page_size) return ASPD_ERR_BAD_DESCRIPTOR;
      regs.push_back({q.tail_off, q.tail_off + q.tail_len});
    }
    for (const Region& g : regs)
      if (g.hi > cap) return ASPD_ERR_BAD_DESCRIPTOR;
    std::vector<Region> sorted;
    for (const Region& g : regs)
      if (g.hi > g.lo) sorted.push_back(g);
    std::sort(sorted.begin(), sorted.end(), [](const Region& a, const Region& b) { return a.lo < b.lo; });
    for (size_t i = 1; i < sorted.size(); ++i)
      if (sorted[i].lo < sorted[i - 1].hi) return ASPD_ERR_BAD_DESCRIPTOR;
    for (int p = 0; p < q.n_pages; ++p) {
      int32_t id = page_ids[q.page_begin + p];
      if (id < 0 || id >= n_pool_pages) return ASPD_ERR_BAD_DESCRIPTOR;
      if (used[id]) return ASPD_ERR_BAD_DESCRIPTOR;
      used[id] = 1;
    }
  }
  return ASPD_OK;
}

}  // namespace

extern "C" {

const char* aspd_strerror(int status) {
  switch (status) {
    case ASPD_OK: return "ok";
    case ASPD_ERR_INVALID_ARG: return "invalid argument";
    case ASPD_ERR_BAD_DESCRIPTOR: return "bad descriptor (overlap, out-of-table slot, alignment, q_len > kv_len or page id)";
    case ASPD_ERR_UNSUPPORTED: return "unsupported shape (head_dim, page_size or dtype)";
    case ASPD_ERR_CUDA: return "CUDA runtime or launch error";
    case ASPD_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case ASPD_ERR_NOMEM: return "out of memory";
    case ASPD_ERR_TOO_LARGE: return "size exceeds a stated maximum";
    default: return "unknown status";
  }
}

size_t aspd_pool_bytes(const aspd_shape_t* shape, int64_t n_pages) {
  if (check_shape(shape) != ASPD_OK || n_pages < 0) return 0;
  return (size_t)n_pages * shape->n_kv_heads * tile_bytes(shape->page_size, shape->head_dim, esize_of(shape->dtype));
}

int aspd_count_new_tokens(const aspd_request_t* req, const aspd_branch_t* br, int n_req, int mode) {
  int rc = check_counts(req, br, n_req, mode);
  if (rc != ASPD_OK) return rc;
  long n = 0;
  for (int r = 0; r < n_req; ++r) {
    if (mode == ASPD_MODE_SERIAL) { ++n; continue; }
    for (int b = 0; b < req[r].n_branches; ++b) n += std::max(0, br[req[r].branch_begin + b].q_len);
  }
  if (n > (1 << 24)) return ASPD_ERR_TOO_LARGE;
  return (int)n;
}

int aspd_positions(const aspd_request_t* req, const aspd_branch_t* br, int n_req, int mode, int32_t* pos_out,
                   int32_t* slot_out, int32_t* req_out) {
  int n = aspd_count_new_tokens(req, br, n_req, mode);
  if (n < 0) return n;
  if (n > 0 && (!pos_out || !slot_out)) return ASPD_ERR_INVALID_ARG;
  int t = 0;
  for (int r = 0; r < n_req; ++r) {
    const aspd_request_t& q = req[r];
    if (mode == ASPD_MODE_BRANCH) {
      // Eq. 4, stage_start: every token cached before the stage counts -- the prefix and the regions
      // of earlier stages (merged branches, serial tokens between stages); all branches share it
      long stage_start = q.prefix_len;
      for (int b = 0; b < q.n_branches; ++b)
        if (br[q.branch_begin + b].q_len == ASPD_Q_SHARED) stage_start += br[q.branch_begin + b].kv_len;
      for (int b = 0; b < q.n_branches; ++b) {
        const aspd_branch_t& x = br[q.branch_begin + b];
        const long first = x.pos_start == ASPD_POS_AUTO ? stage_start : (long)x.pos_start;
        for (int i = 0; i < x.q_len; ++i, ++t) {
          int k = x.kv_len - x.q_len + i;        // index of the token inside its branch
          if (first + k > INT32_MAX) return ASPD_ERR_TOO_LARGE;
          pos_out[t] = (int32_t)(first + k);     // Eq. 4: stage_start + delta
          slot_out[t] = x.kv_off + k;
          if (req_out) req_out[t] = r;
        }
      }
    } else {
      long total = q.prefix_len;                  // Eq. 4, main branch: every cached token counts
      for (int b = 0; b < q.n_branches; ++b) total += br[q.branch_begin + b].kv_len;
      pos_out[t] = (int32_t)(total + q.tail_len - 1);
      slot_out[t] = q.tail_off + q.tail_len - 1;
      if (req_out) req_out[t] = r;
      ++t;
    }
  }
  return ASPD_OK;
}

int aspd_visible_slots(const aspd_request_t* req, const aspd_branch_t* br, int n_req, int mode, int n_slots,
                       uint8_t* vis_out) {
  return aspd_visible_slots_masked(req, br, n_req, mode, ASPD_MASK_BRANCH_INVISIBLE, n_slots, vis_out);
}

int aspd_visible_slots_masked(const aspd_request_t* req, const aspd_branch_t* br, int n_req, int mode, int mask, int n_slots,
                              uint8_t* vis_out) {
  int n = aspd_count_new_tokens(req, br, n_req, mode);
  if (n < 0) return n;
  if (!vis_out || n_slots < 0 || (mask != ASPD_MASK_BRANCH_INVISIBLE && mask != ASPD_MASK_SHARED)) return ASPD_ERR_INVALID_ARG;
  memset(vis_out, 0, (size_t)n * n_slots);
  int t = 0;
  auto mark = [&](int tok, int lo, int hi) -> int {
    if (hi > n_slots) return ASPD_ERR_INVALID_ARG;
    for (int s = lo; s < hi; ++s) vis_out[(size_t)tok * n_slots + s] = 1;
    return ASPD_OK;
  };
  for (int r = 0; r < n_req; ++r) {
    const aspd_request_t& q = req[r];
    if (mode == ASPD_MODE_BRANCH) {
      for (int b = 0; b < q.n_branches; ++b) {
        const aspd_branch_t& x = br[q.branch_begin + b];
        for (int i = 0; i < x.q_len; ++i, ++t) {
          if (mark(t, 0, q.prefix_len)) return ASPD_ERR_INVALID_ARG;
          for (int s2 = 0; s2 < q.n_branches; ++s2) {          // regions of earlier stages (Eq. 3, third case)
            const aspd_branch_t& y = br[q.branch_begin + s2];
            if (y.q_len == ASPD_Q_SHARED && mark(t, y.kv_off, y.kv_off + y.kv_len)) return ASPD_ERR_INVALID_ARG;
          }
          const int k = x.kv_len - x.q_len + i;                // the token's offset in its branch
          if (mark(t, x.kv_off, x.kv_off + k + 1)) return ASPD_ERR_INVALID_ARG;
          if (mask == ASPD_MASK_SHARED)                         // smaller offsets of the stage's other branches
            for (int s2 = 0; s2 < q.n_branches; ++s2) {
              const aspd_branch_t& y = br[q.branch_begin + s2];
              if (s2 != b && y.q_len != ASPD_Q_SHARED && mark(t, y.kv_off, y.kv_off + std::min(k, y.kv_len))) return ASPD_ERR_INVALID_ARG;
            }
        }
      }
    } else {
      if (mark(t, 0, q.prefix_len)) return ASPD_ERR_INVALID_ARG;
      for (int b = 0; b < q.n_branches; ++b) {
        const aspd_branch_t& x = br[q.branch_begin + b];
        if (mark(t, x.kv_off, x.kv_off + x.kv_len)) return ASPD_ERR_INVALID_ARG;
      }
      if (mark(t, q.tail_off, q.tail_off + q.tail_len)) return ASPD_ERR_INVALID_ARG;
      ++t;
    }
  }
  return ASPD_OK;
}

static int plan_to_device(aspd_plan* p, cudaStream_t s);

// sm_count_override > 0: plan for a grid of that many SMs without asking the device (aspd_plan_update
// re-plans on the host for the device the plan already lives on)
static int plan_create_impl(const aspd_shape_t* shape, const aspd_request_t* req, const aspd_branch_t* br,
                            const int32_t* page_ids, int n_req, int64_t n_pool_pages, int mode, const int32_t* q_pos,
                            const aspd_tuning_t* tuning, void* stream, int sm_count_override, aspd_plan_t** plan_out) {
  if (!plan_out) return ASPD_ERR_INVALID_ARG;
  *plan_out = nullptr;
  int rc = check_shape(shape);
  if (rc) return rc;
  rc = check_counts(req, br, n_req, mode);
  if (rc) return rc;
  rc = check_layout(shape, req, br, page_ids, n_req, n_pool_pages, mode);
  if (rc) return rc;
  const int n_new = aspd_count_new_tokens(req, br, n_req, mode);
  if (n_new < 0) return n_new;

  aspd_tuning_t tune = {ASPD_KERNEL_AUTO, 0, 0, 0, 0, ASPD_MASK_BRANCH_INVISIBLE, 0, ASPD_COMBINE_AUTO, 0, 0};
  if (tuning) tune = *tuning;
  const int ps = shape->page_size, d = shape->head_dim, Hq = shape->n_q_heads, Hkv = shape->n_kv_heads;
  const int G = Hq / Hkv, es = esize_of(shape->dtype);
  if (tune.chunk_tokens < 0 || tune.chunk_tokens % ps || tune.n_ctas < 0) return ASPD_ERR_INVALID_ARG;
  if (tune.mask != ASPD_MASK_BRANCH_INVISIBLE && tune.mask != ASPD_MASK_SHARED) return ASPD_ERR_INVALID_ARG;
  if (tune.wide_rows != 0 && tune.wide_rows != 128 && tune.wide_rows != 256) return ASPD_ERR_INVALID_ARG;
  if (tune.mma_m != 0 && tune.mma_m != 64 && tune.mma_m != 96 && tune.mma_m != 128) return ASPD_ERR_INVALID_ARG;
  if (tune.combine != ASPD_COMBINE_AUTO && tune.combine != ASPD_COMBINE_KERNEL && tune.combine != ASPD_COMBINE_FUSED) return ASPD_ERR_INVALID_ARG;
  const bool shared_mask = tune.mask == ASPD_MASK_SHARED && mode == ASPD_MODE_BRANCH;
  const bool mma_ok = shape->dtype == ASPD_DTYPE_BF16 && d == 128 && ps == 16;
  int kernel = tune.kernel;
  if (kernel == ASPD_KERNEL_AUTO) kernel = mma_ok ? ASPD_KERNEL_MMA : ASPD_KERNEL_GENERIC;
  if (kernel == ASPD_KERNEL_MMA && !mma_ok) return ASPD_ERR_UNSUPPORTED;
  if (kernel != ASPD_KERNEL_MMA && kernel != ASPD_KERNEL_GENERIC) return ASPD_ERR_INVALID_ARG;

  aspd_plan* p = new (std::nothrow) aspd_plan();
  if (!p) return ASPD_ERR_NOMEM;
  p->shape = *shape; p->mode = mode; p->n_req = n_req; p->n_new = n_new; p->kernel = kernel;
  p->stable_cache = tune.stable_cache ? 1 : 0;
  p->shared_mask = (tune.mask == ASPD_MASK_SHARED && mode == ASPD_MODE_BRANCH) ? 1 : 0;
  p->host_only = tune.host_only; p->n_pool_pages = n_pool_pages; p->device_base = nullptr; p->device_bytes = 0;
  memset(&p->dev, 0, sizeof(p->dev));
  p->tune = tune;
  p->sm_count = sm_count_override > 0 ? sm_count_override : 148;
  if (!tune.host_only && sm_count_override <= 0) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      delete p; return ASPD_ERR_CUDA;
    }
    p->sm_count = sms;
  }

  // ---- new-token table --------------------------------------------------------------
  std::vector<int32_t> pos(n_new), slot(n_new), treq(n_new), tok_page(n_new), tok_row(n_new);
  rc = aspd_positions(req, br, n_req, mode, pos.data(), slot.data(), treq.data());
  if (rc) { delete p; return rc; }
  for (int t = 0; t < n_new; ++t) {
    tok_page[t] = page_ids[req[treq[t]].page_begin + slot[t] / ps];
    tok_row[t] = slot[t] % ps;
    if (q_pos) { if (q_pos[t] < 0) { delete p; return ASPD_ERR_INVALID_ARG; } pos[t] = q_pos[t]; }
  }

  // ---- key streams -------------------------------------------------------------------
  // Per request, the pages the step must read, in one sequence: the prefix, then every branch
  // that has queries (branch mode) or every branch and the tail (serial mode).  Each entry is
  // (physical page, valid rows); the padding rows of partly filled pages are masked by the
  // kernels.  A new token sees stream keys [0, pe) (the prefix) and [lo, hi) (its own branch up
  // to itself); a serial token sees the whole stream.
  // With block_tok > 0 (plans that deal whole streams) every run of block_tok query tokens of a
  // request gets a sequence of its own: the prefix and, of the branches, only the pages that one
  // of the run's tokens can see.
  const int max_tok = std::max(1, kMaxRowsPerItem / G);
  struct Block { int request, tok0, n_tok, visit0, n_pages; };
  std::vector<int2> visit;
  std::vector<Block> blocks;
  std::vector<int4> tok_vis(n_new);
  int64_t kv_tokens = 0;
  const bool tok_field_fits = n_new < (1 << 18);      // the 18 bits above bit 13 of a page entry hold a token index
  auto build_visit = [&](int block_tok) {
    visit.clear(); blocks.clear();
    int64_t kv_count = 0;
    int t = 0;
    // new_key0 / new_tok0: the keys [new_key0, len) of the region are this step's new tokens
    // new_tok0, new_tok0 + 1, ...; a page entry carries (valid rows | new rows << 8 | first new
    // token << 13) so that a fused step can write those rows just before it reads the page.
    // Under the shared mask the upper bits carry the page's index inside its branch instead (its
    // first key's offset / page_size; such plans never fuse the append): a token at offset k
    // also sees the keys of other branches whose offset is below k.
    auto push_region = [&](const aspd_request_t& q, int slot0, int len, int new_key0, int new_tok0, bool branch_pages = false) {
      for (int s0 = 0; s0 < len; s0 += ps) {
        const int nv = std::min(ps, len - s0), first_new = std::max(s0, new_key0);
        const int n_newrows = std::max(0, s0 + nv - first_new);
        int y = nv;
        if (n_newrows > 0) y |= (std::min(n_newrows, 31) << 8);   // 5 bits; a count is only needed where pages have 16 rows
        if (shared_mask) y |= branch_pages ? (s0 / ps) << 13 : 0;
        else if (n_newrows > 0 && tok_field_fits) y |= (new_tok0 + first_new - new_key0) << 13;
        visit.push_back(make_int2(page_ids[q.page_begin + (slot0 + s0) / ps], y));
      }
    };
    auto push_shared = [&](const aspd_request_t& q) {            // prefix and regions of earlier stages: seen by every branch
      push_region(q, 0, q.prefix_len, q.prefix_len, 0);
      for (int b = 0; b < q.n_branches; ++b) {
        const aspd_branch_t& x = br[q.branch_begin + b];
        if (x.q_len == ASPD_Q_SHARED) push_region(q, x.kv_off, x.kv_len, x.kv_len, 0);
      }
    };
    for (int r = 0; r < n_req; ++r) {
      const aspd_request_t& q = req[r];
      const int t_req = t, v0 = (int)visit.size();
      if (mode == ASPD_MODE_BRANCH) {
        int nq = 0;
        int64_t kv_req = q.prefix_len;                         // keys of this request that the step reads
        for (int b = 0; b < q.n_branches; ++b) {
          const aspd_branch_t& x = br[q.branch_begin + b];
          nq += std::max(0, x.q_len);
          if (x.q_len != 0 || shared_mask) kv_req += x.kv_len;
        }
        if (nq == 0) continue;
        kv_count += kv_req;
        if (block_tok == 0) {
          push_shared(q);
          const int pe = ((int)visit.size() - v0) * ps;
          for (int b = 0; b < q.n_branches; ++b) {
            const aspd_branch_t& x = br[q.branch_begin + b];
            if (x.q_len < 0 || (x.q_len == 0 && !shared_mask)) continue;     // shared mask: also branches without queries
            const int lo = ((int)visit.size() - v0) * ps, prior = x.kv_len - x.q_len;
            push_region(q, x.kv_off, x.kv_len, prior, t, true);
            for (int i = 0; i < x.q_len; ++i) tok_vis[t++] = make_int4(pe, lo, lo + prior + i + 1, shared_mask ? prior + i : 0);
          }
          blocks.push_back({r, t_req, nq, v0, (int)visit.size() - v0});
        } else {
          for (int blk0 = 0; blk0 < nq; blk0 += block_tok) {
            const int blk1 = std::min(nq, blk0 + block_tok), bv0 = (int)visit.size();
            push_shared(q);
            const int pe = ((int)visit.size() - bv0) * ps;
            int off = 0;                                       // index, among the request's new tokens, of the branch's first
            for (int b = 0; b < q.n_branches; ++b) {
              const aspd_branch_t& x = br[q.branch_begin + b];
              if (x.q_len <= 0) continue;
              const int a = std::max(blk0, off), e = std::min(blk1, off + x.q_len);
              if (a < e) {
                const int lo = ((int)visit.size() - bv0) * ps, prior = x.kv_len - x.q_len;
                push_region(q, x.kv_off, prior + (e - off), prior, t_req + off);   // up to the run's last token of this branch
                for (int i = a - off; i < e - off; ++i) tok_vis[t_req + off + i] = make_int4(pe, lo, lo + prior + i + 1, 0);
              }
              off += x.q_len;
            }
            blocks.push_back({r, t_req + blk0, blk1 - blk0, bv0, (int)visit.size() - bv0});
          }
          t += nq;
        }
      } else {
        push_region(q, 0, q.prefix_len, q.prefix_len, 0);
        kv_count += q.prefix_len + q.tail_len;
        for (int b = 0; b < q.n_branches; ++b) {
          const aspd_branch_t& x = br[q.branch_begin + b];
          push_region(q, x.kv_off, x.kv_len, x.kv_len, 0);
          kv_count += x.kv_len;
        }
        push_region(q, q.tail_off, q.tail_len, q.tail_len - 1, t);
        tok_vis[t++] = make_int4(kCausalAll, 0, 0, 0);
        blocks.push_back({r, t_req, 1, v0, (int)visit.size() - v0});
      }
    }
    kv_tokens = kv_count;
  };
  build_visit(0);

  // ---- work items: a contiguous, equal share of all pages for every CTA -----------------
  // Streams are walked in the order (request, row block, KV head); the concatenation of all
  // streams is cut at the CTA boundaries (and, if asked for, every chunk_tokens keys).
  struct Stream { int request, tok0, n_tok, head, page0, n_pages, row_block; };
  std::vector<int2> row_blocks;
  std::vector<Stream> streams;
  long total_pages = 0;
  auto build_streams = [&](int tok_per_block) {
    row_blocks.clear(); streams.clear(); total_pages = 0;
    for (const Block& bk : blocks) {
      if (bk.n_tok == 0 || bk.n_pages == 0) continue;
      for (int i0 = 0; i0 < bk.n_tok; i0 += tok_per_block) {
        row_blocks.push_back(make_int2(bk.tok0 + i0, std::min(tok_per_block, bk.n_tok - i0)));
        for (int h = 0; h < Hkv; ++h) {
          streams.push_back({bk.request, bk.tok0 + i0, std::min(tok_per_block, bk.n_tok - i0), h, bk.visit0, bk.n_pages,
                             (int)row_blocks.size() - 1});
          total_pages += bk.n_pages;
        }
      }
    }
  };
  build_streams(max_tok);
  auto ctas_for = [&](long pages) {
    const int want = tune.n_ctas > 0 ? tune.n_ctas : p->sm_count;
    // do not cut finer than one 128-key tile per CTA (measured on a 2.5 k-token step: 80 CTAs with a
    // full tile each take 10.6 us per layer, 148 CTAs with half a tile 11.9: fewer records to combine)
    return (int)std::max(1L, std::min((long)want, (pages + 7) / 8));
  };
  // With many more streams than CTAs (a step with many query tokens per branch: masked prefill,
  // teacher forcing) nothing is cut: every stream is one item, and the streams are dealt to the
  // CTAs in turn, longest requests first, so that at any moment all CTAs read the K/V pages of the
  // same one or two requests (which then stay in L2) and every CTA gets one stream of each round.
  // Every row block then gets a page sequence of its own, without the branch pages none of its
  // tokens sees, and the tensor-core kernel takes row blocks of up to 128 rows (its wide variant).
  // (only where the step fills the grid, or the caller chose the grid: a step of a few pages has few CTAs and many streams by default)
  bool deal_streams = mode == ASPD_MODE_BRANCH && !shared_mask && tune.chunk_tokens == 0 &&
                      (long)streams.size() >= 4L * ctas_for(total_pages) && (tune.n_ctas > 0 || ctas_for(total_pages) >= p->sm_count);
  p->wide = 0;
  if (deal_streams) {
    p->wide = (kernel == ASPD_KERNEL_MMA && kMaxRowsWide / G > max_tok) ? 1 : 0;
    // A step in which some request has more query tokens than one 128-row tile holds takes row blocks
    // of two tiles (the two-tile variant of the kernel: both tiles are scored against every K/V tile
    // the CTA fetches, one softmax group per tile), unless the caller asked for single tiles.
    if (p->wide && tune.wide_rows != 128) {
      int most_q = 0;
      for (const Block& bk : blocks) most_q = std::max(most_q, bk.n_tok);
      if (most_q > kMaxRowsWide / G || tune.wide_rows == 256) p->wide = 2;
    }
    const int tok_per_block = p->wide ? p->wide * (kMaxRowsWide / G) : max_tok;
    build_visit(tok_per_block);
    build_streams(tok_per_block);
  }
  const int n_ctas = ctas_for(total_pages);
  const int chunk_pages = tune.chunk_tokens > 0 ? tune.chunk_tokens / ps : (1 << 28);
  p->chunk_tokens = tune.chunk_tokens; p->n_ctas = n_ctas;
  std::vector<int32_t> n_parts((size_t)n_new * Hkv, 0), part_base((size_t)n_new * Hkv + 1, 0), cta_item0(n_ctas + 1, 0);
  p->dealt = deal_streams ? 1 : 0;
  if (deal_streams) {
    std::vector<int> order(streams.size());
    for (size_t i = 0; i < order.size(); ++i) order[i] = (int)i;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return streams[a].n_pages > streams[b].n_pages; });
    std::vector<std::vector<int>> mine(n_ctas);
    for (size_t i = 0; i < order.size(); ++i) {
      const int round = (int)(i / n_ctas), k = (int)(i % n_ctas);
      mine[(round & 1) ? n_ctas - 1 - k : k].push_back(order[i]);       // back and forth: evens out the rounds
    }
    for (int c = 0; c < n_ctas; ++c) {
      cta_item0[c] = (int)p->items.size();
      for (int si : mine[c]) {
        const Stream& st = streams[si];
        DeviceItem it;
        it.q_tok0 = st.tok0; it.n_q_tok = st.n_tok; it.kv_head = st.head; it.page0 = st.page0; it.n_pages = st.n_pages;
        it.key0 = 0; it.part_slot = 0; it.request = st.request; it.row_block = st.row_block; it.n_parts = 1;
        p->items.push_back(it);
        for (int i = 0; i < st.n_tok; ++i) n_parts[(size_t)(st.tok0 + i) * Hkv + st.head] = 1;
      }
    }
    cta_item0[n_ctas] = (int)p->items.size();
  } else {
    // Every CTA gets the same cost, cost = pages + kItemCost per item it starts: an item boundary
    // (new query tile, ragged last tile, epilogue) costs about as much as streaming a dozen pages,
    // so CTAs that end up with several short items get fewer pages.
    const double kItemCost = 12.0;
    // a page costs a little more the more query rows are scored against it (best measured balance:
    // 0.35 % per row), so streams of requests with many branches weigh more
    const double kRowCost = 0.0035;
    auto page_cost = [&](const Stream& st) { return 1.0 + kRowCost * st.n_tok * G; };
    // the share is re-derived from what is left whenever a CTA is closed, so rounding does not pile up
    double cost_left = 0.0;
    for (const Stream& st : streams) cost_left += page_cost(st) * st.n_pages;
    long streams_left = (long)streams.size();
    auto share_now = [&](int ctas_left) {
      return (cost_left + kItemCost * ((double)streams_left + ctas_left)) / std::max(1, ctas_left);
    };
    double share = share_now(n_ctas);
    int cta = 0;
    double acc = 0.0;                              // cost already given to the current CTA
    auto next_cta = [&]() { cta_item0[++cta] = (int)p->items.size(); acc = 0.0; share = share_now(n_ctas - cta); };
    for (const Stream& st : streams) {
      int at = 0, slot = 0;
      const size_t first_item = p->items.size();
      const double pc = page_cost(st);
      --streams_left;
      while (at < st.n_pages) {
        double room = (share - acc - kItemCost) / pc;   // pages that still fit if an item starts here
        if (room < 1.0 && acc > 0.0 && cta + 1 < n_ctas) { next_cta(); continue; }
        long take = std::min<long>(st.n_pages - at, chunk_pages);
        if (cta + 1 < n_ctas) take = std::min<long>(take, std::max<long>(1, (long)(room + 0.5)));
        // a cut inside a stream goes on a tile boundary (8 pages) where the item is long enough: the item's
        // last tile is then a full one (measured on the serving mix: 0.4 % on the step)
        if (take < st.n_pages - at && tune.chunk_tokens == 0 && ps == 16 && take >= 12)
          take = std::min<long>((take + 4) / 8 * 8, st.n_pages - at);
        DeviceItem it;
        it.q_tok0 = st.tok0; it.n_q_tok = st.n_tok; it.kv_head = st.head; it.page0 = st.page0 + at;
        it.n_pages = (int)take; it.key0 = at * ps; it.part_slot = slot++; it.request = st.request;
        it.row_block = st.row_block; it.n_parts = 0;
        p->items.push_back(it);
        at += (int)take;
        cost_left -= pc * take;
        acc += kItemCost + pc * (double)take;
        if (acc >= share - 0.5 && cta + 1 < n_ctas) next_cta();
      }
      for (int i = 0; i < st.n_tok; ++i) n_parts[(size_t)(st.tok0 + i) * Hkv + st.head] = slot;
      for (size_t i = first_item; i < p->items.size(); ++i) p->items[i].n_parts = slot;
    }
    while (cta < n_ctas) cta_item0[++cta] = (int)p->items.size();
  }
  // rows that are new this step, per CTA: what a fused step must write before the CTA reads
  std::vector<int4> dirty;
  std::vector<int32_t> cta_dirty0(n_ctas + 1, 0);
  for (int c = 0; c < n_ctas; ++c) {
    cta_dirty0[c] = (int)dirty.size();
    for (int i = cta_item0[c]; i < cta_item0[c + 1] && !shared_mask; ++i) {
      const DeviceItem& it = p->items[i];
      for (int pg = 0; pg < it.n_pages; ++pg) {
        const int2 v = visit[it.page0 + pg];
        const int cnt = (v.y >> 8) & 31, tok0 = v.y >> 13, row0 = (v.y & 255) - cnt;
        for (int k = 0; k < cnt; ++k) dirty.push_back(make_int4(v.x, it.kv_head, tok0 + k, row0 + k));
      }
    }
  }
  cta_dirty0[n_ctas] = (int)dirty.size();
  {
    // the fused step writes a CTA's new rows in batches at the start of the kernel; with many new
    // rows per CTA (a branch-open step) the separate append kernel is the faster way
    int most = 0;
    for (int c = 0; c < n_ctas; ++c) most = std::max(most, cta_dirty0[c + 1] - cta_dirty0[c]);
    p->fuse_append = (most <= 20 && !shared_mask && tok_field_fits && p->wide != 2) ? 1 : 0;
  }
  // the merge of a token's records inside the attention kernel: stream-K plans of the tensor-core kernel
  // 1: both MMAs with M = 64; 2: only P.V (the default: at most 64 of P.V's 128 rows are ever read, a quarter
  // less tensor work lifts the power-capped clock and the softmax layout, which M = 64 scores would slow
  // down, stays as it is); 0: both with M = 128
  p->m64 = (kernel == ASPD_KERNEL_MMA && !deal_streams) ? (tune.mma_m == 64 ? 1 : tune.mma_m == 128 ? 0 : 2) : 0;
  p->stagger_start = (!deal_streams && total_pages <= 6L * 8 * n_ctas) ? 1 : 0;       // at most six 128-key tiles per CTA
  // Merging inside the attention kernel is an option, not the default.  Measured on every workload of
  // the benchmark, the CTA that stores a pair's last record is a CTA at the very end of its own work,
  // so its fence, count and merge (1.5 us + one memory round trip per 16 rows of the pairs it ended
  // up with; all rows of a stream cut into dozens of parts land on one CTA) lengthen the kernel by
  // more than the combine launch costs, whose blocks are resident and waiting when the pass ends.
  p->single_launch = (kernel == ASPD_KERNEL_MMA && !deal_streams && tune.combine == ASPD_COMBINE_FUSED) ? 1 : 0;
  for (size_t i = 0; i < n_parts.size(); ++i) part_base[i + 1] = part_base[i] + n_parts[i];
  p->n_items = (int)p->items.size();
  p->n_partials = part_base[n_parts.size()];
  p->kv_tokens_read = kv_tokens;
  p->algorithmic_bytes = 2LL * Hkv * d * es * kv_tokens + 2LL * es * Hq * d * n_new + 2LL * Hkv * d * es * n_new;
  p->visit = visit;
  p->n_row_blocks = (int)row_blocks.size();
  p->cta_item0 = cta_item0; p->part_base = part_base; p->row_blocks = row_blocks; p->q_pos = pos;
  p->tok_vis = tok_vis;
  p->tok_page = tok_page; p->tok_row = tok_row; p->dirty = dirty; p->cta_dirty0 = cta_dirty0;
  if (tune.host_only) { *plan_out = p; return ASPD_OK; }
  rc = plan_to_device(p, (cudaStream_t)stream);
  if (rc) { delete p; return rc; }
  *plan_out = p;
  return ASPD_OK;
}

int aspd_plan_create(const aspd_shape_t* shape, const aspd_request_t* req, const aspd_branch_t* br,
                     const int32_t* page_ids, int n_req, int64_t n_pool_pages, int mode, const int32_t* q_pos,
                     const aspd_tuning_t* tuning, void* stream, aspd_plan_t** plan_out) {
  return plan_create_impl(shape, req, br, page_ids, n_req, n_pool_pages, mode, q_pos, tuning, stream, 0, plan_out);
}

// ---- one device allocation, one staging blob ----------------------------------------------
// Offsets of the plan's tables inside its device block.  The tables whose size depends on the
// lengths of the step (items, page list, new-row list, partial records) get `slack` times the room
// they need now, so that aspd_plan_update can re-plan into the same addresses.
static void plan_layout(const aspd_plan* p, double slack, aspd::PlanLayout* L) {
  const aspd_shape_t& sh = p->shape;
  const int d = sh.head_dim, Hq = sh.n_q_heads, Hkv = sh.n_kv_heads, G = Hq / Hkv, es = esize_of(sh.dtype), n_new = p->n_new;
  auto cap = [&](size_t n) { return std::max<size_t>(1, (size_t)((double)n * slack) + (slack > 1.0 ? 64 : 0)); };
  L->cap_items = cap(p->items.size()); L->cap_visit = cap(p->visit.size()); L->cap_dirty = cap(p->dirty.size());
  L->cap_partials = cap((size_t)p->n_partials);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  L->o_items = take(sizeof(DeviceItem) * L->cap_items);
  L->o_cta = take(sizeof(int4) * std::max(1, p->n_ctas));
  L->o_visit = take(sizeof(int2) * L->cap_visit);
  L->o_cdirty = take(sizeof(int32_t) * (p->n_ctas + 1));
  L->o_dirty = take(sizeof(int4) * L->cap_dirty);
  L->o_tpage = take(sizeof(int32_t) * std::max(1, n_new));
  L->o_trow = take(sizeof(int32_t) * std::max(1, n_new));
  L->o_tpos = take(sizeof(int32_t) * std::max(1, n_new));
  L->o_tvis = take(sizeof(int4) * std::max(1, n_new));
  L->o_rb = take(sizeof(int2) * std::max<size_t>(1, p->row_blocks.size()));
  L->o_pbase = take(sizeof(int32_t) * p->part_base.size());
  L->o_freq = take(sizeof(double) * (d / 2));
  L->upload_bytes = off;
  // the status word is zeroed when the plan is created and never uploaded again, so that a time-out
  // recorded by an earlier launch survives aspd_plan_update until aspd_plan_status reads it
  L->o_status = take(sizeof(int32_t) * 2);
  L->o_arrive = take(sizeof(int32_t) * std::max(1, n_new) * Hkv);   // right behind the status word: cleared with it
  L->o_qcs = take(sizeof(float2) * std::max(1, n_new) * (d / 2));   // filled on the device from tok_pos and inv_freq
  L->o_wso = take(sizeof(float) * L->cap_partials * G * d);
  L->o_wsml = take(sizeof(float2) * L->cap_partials * G);
  L->o_stq = take((size_t)es * std::max(1, n_new) * Hq * d);
  L->o_stk = take((size_t)es * std::max(1, n_new) * Hkv * d);
  L->o_stv = take((size_t)es * std::max(1, n_new) * Hkv * d);
  L->o_sto = take((size_t)es * std::max(1, n_new) * Hq * d);
  L->o_stp = take(sizeof(int32_t) * std::max(1, n_new));
  L->device_bytes = off;
  L->n_row_blocks = p->row_blocks.size(); L->n_part_base = p->part_base.size();
}

// Assembles the tables in the plan's page-locked buffer, sends them to the device block and fills
// the cos/sin table there.  The caller has made sure that the buffer's previous copy has completed.
static int plan_upload(aspd_plan* p, cudaStream_t s) {
  const aspd::PlanLayout& L = p->layout;
  const int n_new = p->n_new, d = p->shape.head_dim, n_ctas = p->n_ctas;
  uint8_t* blob = static_cast<uint8_t*>(p->host_block);
  memset(blob, 0, L.upload_bytes);
  if (!p->items.empty()) memcpy(blob + L.o_items, p->items.data(), sizeof(DeviceItem) * p->items.size());
  fill_cta_head(p, reinterpret_cast<int4*>(blob + L.o_cta));
  if (!p->visit.empty()) memcpy(blob + L.o_visit, p->visit.data(), sizeof(int2) * p->visit.size());
  memcpy(blob + L.o_cdirty, p->cta_dirty0.data(), sizeof(int32_t) * (n_ctas + 1));
  if (!p->dirty.empty()) memcpy(blob + L.o_dirty, p->dirty.data(), sizeof(int4) * p->dirty.size());
  if (n_new) {
    memcpy(blob + L.o_tpage, p->tok_page.data(), sizeof(int32_t) * n_new);
    memcpy(blob + L.o_trow, p->tok_row.data(), sizeof(int32_t) * n_new);
    memcpy(blob + L.o_tpos, p->q_pos.data(), sizeof(int32_t) * n_new);
    memcpy(blob + L.o_tvis, p->tok_vis.data(), sizeof(int4) * n_new);
  }
  if (!p->row_blocks.empty()) memcpy(blob + L.o_rb, p->row_blocks.data(), sizeof(int2) * p->row_blocks.size());
  memcpy(blob + L.o_pbase, p->part_base.data(), sizeof(int32_t) * p->part_base.size());
  double* freq = reinterpret_cast<double*>(blob + L.o_freq);
  for (int i = 0; i < d / 2; ++i) freq[i] = pow((double)p->shape.rope_theta, -2.0 * i / d);
  if (cudaMemcpyAsync(p->device_base, blob, L.upload_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return ASPD_ERR_CUDA;
  if (p->upload_done) { cudaEventDestroy(p->upload_done); p->upload_done = nullptr; }
  if (cudaEventCreateWithFlags(&p->upload_done, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventRecord(p->upload_done, s) != cudaSuccess) {
    if (p->upload_done) cudaEventDestroy(p->upload_done);
    p->upload_done = nullptr;
    cudaStreamSynchronize(s);                      // no event to tell when the buffer is free again: be done with it now
  }
  if (std::find(p->streams.begin(), p->streams.end(), s) == p->streams.end()) p->streams.push_back(s);
  // cos/sin of every new token's position (query rotation, fused append): on the device, after the upload
  return n_new > 0 ? launch_qcs(p, s) : ASPD_OK;
}

static int plan_to_device(aspd_plan* p, cudaStream_t s) {
  plan_layout(p, p->tune.updatable ? 1.25 : 1.0, &p->layout);
  const aspd::PlanLayout& L = p->layout;
  p->device_bytes = L.device_bytes;
  void* base = nullptr;
  int rc = block_acquire(L.device_bytes, L.upload_bytes, s, &base, &p->block_bytes, &p->host_block, &p->host_block_bytes);
  if (rc) return rc;
  uint8_t* b8 = (uint8_t*)base;
  p->device_base = base;
  p->dev.items = (const DeviceItem*)(b8 + L.o_items);
  p->dev.cta_head = (const int4*)(b8 + L.o_cta);
  p->dev.visit = (const int2*)(b8 + L.o_visit);
  p->dev.cta_dirty0 = (const int32_t*)(b8 + L.o_cdirty);
  p->dev.dirty = (const int4*)(b8 + L.o_dirty);
  p->dev.tok_vis = (const int4*)(b8 + L.o_tvis);
  p->dev.row_blocks = (const int2*)(b8 + L.o_rb);
  p->dev.tok_page = (const int32_t*)(b8 + L.o_tpage);
  p->dev.tok_row = (const int32_t*)(b8 + L.o_trow);
  p->dev.tok_pos = (const int32_t*)(b8 + L.o_tpos);
  p->dev.q_cs = (const float2*)(b8 + L.o_qcs);
  p->dev.part_base = (const int32_t*)(b8 + L.o_pbase);
  p->dev.inv_freq = (const double*)(b8 + L.o_freq);
  p->dev.status = (int32_t*)(b8 + L.o_status);
  p->dev.work_counter = p->dev.status + 1;
  p->dev.arrive = (int32_t*)(b8 + L.o_arrive);
  p->dev.ws_o = (float*)(b8 + L.o_wso);
  p->dev.ws_ml = (float2*)(b8 + L.o_wsml);
  p->dev.st_q = b8 + L.o_stq; p->dev.st_k = b8 + L.o_stk; p->dev.st_v = b8 + L.o_stv; p->dev.st_out = b8 + L.o_sto;
  p->dev.st_pos = (int32_t*)(b8 + L.o_stp);
  p->dev.pool_limit = (int32_t)std::min<int64_t>(p->n_pool_pages, INT32_MAX);
  rc = cudaMemsetAsync(p->dev.status, 0, (L.o_arrive - L.o_status) + sizeof(int32_t) * std::max(1, p->n_new) * p->shape.n_kv_heads, s) == cudaSuccess
           ? plan_upload(p, s) : ASPD_ERR_CUDA;
  if (rc) {
    cudaFree(base); cudaFreeHost(p->host_block);
    p->device_base = nullptr; p->host_block = nullptr;
  }
  return rc;
}

int aspd_plan_update(aspd_plan_t* p, const aspd_request_t* req, const aspd_branch_t* br, const int32_t* page_ids, int n_req,
                     const int32_t* q_pos, void* stream) {
  if (!p || p->host_only || !p->device_base) return ASPD_ERR_INVALID_ARG;
  aspd_tuning_t tune = p->tune;
  tune.host_only = 1;
  aspd_plan* t = nullptr;
  int rc = plan_create_impl(&p->shape, req, br, page_ids, n_req, p->n_pool_pages, p->mode, q_pos, &tune, nullptr, p->sm_count, &t);
  if (rc) return rc;
  const aspd::PlanLayout& L = p->layout;
  if (t->n_new != p->n_new || t->n_ctas != p->n_ctas || t->kernel != p->kernel || t->wide != p->wide || t->dealt != p->dealt ||
      t->fuse_append != p->fuse_append || t->shared_mask != p->shared_mask || t->single_launch != p->single_launch || t->m64 != p->m64 || t->kernel != ASPD_KERNEL_MMA ||
      t->row_blocks.size() != L.n_row_blocks || t->part_base.size() != L.n_part_base ||
      (t->algorithmic_bytes >= (128LL << 20)) != (p->algorithmic_bytes >= (128LL << 20))) {   // the combine's launch attribute
    delete t;
    return ASPD_ERR_UNSUPPORTED;
  }
  if (t->items.size() > L.cap_items || t->visit.size() > L.cap_visit || t->dirty.size() > L.cap_dirty ||
      (size_t)t->n_partials > L.cap_partials) {
    delete t;
    return ASPD_ERR_TOO_LARGE;
  }
  // the page-locked buffer is written again: its previous copy must be through
  if (p->upload_done && cudaEventSynchronize(p->upload_done) != cudaSuccess) { delete t; return ASPD_ERR_CUDA; }
  p->n_req = t->n_req; p->n_items = t->n_items; p->n_partials = t->n_partials; p->n_row_blocks = t->n_row_blocks;
  p->kv_tokens_read = t->kv_tokens_read; p->algorithmic_bytes = t->algorithmic_bytes;
  p->items.swap(t->items); p->visit.swap(t->visit); p->tok_vis.swap(t->tok_vis); p->cta_item0.swap(t->cta_item0);
  p->part_base.swap(t->part_base); p->q_pos.swap(t->q_pos); p->row_blocks.swap(t->row_blocks);
  p->tok_page.swap(t->tok_page); p->tok_row.swap(t->tok_row); p->cta_dirty0.swap(t->cta_dirty0); p->dirty.swap(t->dirty);
  delete t;
  return plan_upload(p, (cudaStream_t)stream);
}

int aspd_plan_destroy(aspd_plan_t* plan) {
  if (!plan) return ASPD_OK;
  int rc = ASPD_OK;
  if (plan->device_base) rc = block_release(plan->device_base, plan->block_bytes, plan->host_block, plan->host_block_bytes, plan->upload_done, plan->streams);
  delete plan;
  return rc;
}

int aspd_release_cached_memory(void) { return block_cache_clear(); }

int aspd_plan_info(const aspd_plan_t* p, aspd_plan_info_t* info) {
  if (!p || !info) return ASPD_ERR_INVALID_ARG;
  info->n_new = p->n_new; info->n_items = p->n_items; info->n_partials = p->n_partials;
  info->n_stream_pages = (int32_t)p->visit.size(); info->kernel = p->kernel;
  info->chunk_tokens = p->chunk_tokens; info->n_ctas = p->n_ctas; info->fused_append = (p->kernel == ASPD_KERNEL_MMA && p->fuse_append) ? 1 : 0;
  info->direct_output = attn_mma_direct(p) ? 1 : 0; info->max_rows_per_item = p->wide ? p->wide * kMaxRowsWide : kMaxRowsPerItem;
  info->dealt = p->dealt; info->single_launch = p->single_launch;
  info->mma_m = p->kernel == ASPD_KERNEL_MMA ? (p->m64 == 1 ? 64 : p->m64 == 2 ? 96 : 128) : 0; info->reserved = 0;
  info->workspace_bytes = (int64_t)p->device_bytes;
  info->kv_tokens_read = p->kv_tokens_read; info->algorithmic_bytes = p->algorithmic_bytes;
  return ASPD_OK;
}

int aspd_plan_items(const aspd_plan_t* p, aspd_item_t* items, int max_items) {
  if (!p || (max_items > 0 && !items) || max_items < 0) return ASPD_ERR_INVALID_ARG;
  int n = std::min(max_items, p->n_items);
  static_assert(sizeof(aspd_item_t) == sizeof(DeviceItem) && sizeof(DeviceItem) == 40, "item layouts must match");
  if (n) memcpy(items, p->items.data(), sizeof(DeviceItem) * n);
  return p->n_items;
}

int aspd_plan_cta_ranges(const aspd_plan_t* p, int32_t* first, int max_entries) {
  if (!p || max_entries < 0 || (max_entries > 0 && !first)) return ASPD_ERR_INVALID_ARG;
  const int n = std::min<int>(max_entries, (int)p->cta_item0.size());
  for (int i = 0; i < n; ++i) first[i] = p->cta_item0[i];
  return p->n_ctas;
}

int aspd_plan_stream_pages(const aspd_plan_t* p, int32_t* page_ids, int32_t* n_valid, int max_pages) {
  if (!p || max_pages < 0 || (max_pages > 0 && (!page_ids || !n_valid))) return ASPD_ERR_INVALID_ARG;
  const int n = std::min<int>(max_pages, (int)p->visit.size());
  for (int i = 0; i < n; ++i) { page_ids[i] = p->visit[i].x; n_valid[i] = p->visit[i].y & 255; }
  return (int)p->visit.size();
}

int aspd_plan_token_ranges(const aspd_plan_t* p, int32_t* pe, int32_t* lo, int32_t* hi, int max_tokens) {
  if (!p || max_tokens < 0 || (max_tokens > 0 && (!pe || !lo || !hi))) return ASPD_ERR_INVALID_ARG;
  const int n = std::min<int>(max_tokens, (int)p->tok_vis.size());
  for (int i = 0; i < n; ++i) { pe[i] = p->tok_vis[i].x; lo[i] = p->tok_vis[i].y; hi[i] = p->tok_vis[i].z; }
  return (int)p->tok_vis.size();
}

int aspd_plan_shared_mask_tables(const aspd_plan_t* p, int32_t* below, int32_t* page_in_branch) {
  if (!p || !p->shared_mask || !below || !page_in_branch) return ASPD_ERR_INVALID_ARG;
  for (size_t i = 0; i < p->tok_vis.size(); ++i) below[i] = p->tok_vis[i].w;
  for (size_t i = 0; i < p->visit.size(); ++i) page_in_branch[i] = p->visit[i].y >> 13;
  return ASPD_OK;
}

int aspd_plan_status(aspd_plan_t* p, void* stream) {
  if (!p || p->host_only) return ASPD_ERR_INVALID_ARG;
  int32_t st = 0;
  if (cudaMemcpyAsync(&st, p->dev.status, sizeof(st), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
    return ASPD_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return ASPD_ERR_CUDA;
  return st;
}

int aspd_kv_append(aspd_plan_t* p, const void* k_new, const void* v_new, const int32_t* pos, void* k_pool,
                   void* v_pool, void* stream) {
  if (!p || p->host_only) return ASPD_ERR_INVALID_ARG;
  if (p->n_new == 0) return ASPD_OK;
  if (!k_new || !v_new || !pos || !k_pool || !v_pool || misaligned16(k_new, v_new, k_pool, v_pool)) return ASPD_ERR_INVALID_ARG;
  note_stream(p, stream);
  return launch_append(p, k_new, v_new, pos, k_pool, v_pool, (cudaStream_t)stream);
}

int aspd_attn_partials(aspd_plan_t* p, const void* q, const void* k_pool, const void* v_pool, void* stream) {
  if (!p || p->host_only) return ASPD_ERR_INVALID_ARG;
  if (p->n_new == 0) return ASPD_OK;
  if (!q || !k_pool || !v_pool || misaligned16(q, k_pool, v_pool)) return ASPD_ERR_INVALID_ARG;
  if (p->wide == 2) return ASPD_ERR_UNSUPPORTED;       // the two-tile variant only writes final outputs
  cudaStream_t s = (cudaStream_t)stream;
  note_stream(p, stream);
  return p->kernel == ASPD_KERNEL_MMA ? launch_attn_mma(p, q, k_pool, v_pool, nullptr, s)
                                      : launch_attn_generic(p, q, k_pool, v_pool, s);
}

int aspd_step_partials(aspd_plan_t* p, const void* q, const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                       void* stream) {
  if (!p || p->host_only) return ASPD_ERR_INVALID_ARG;
  if (p->n_new == 0) return ASPD_OK;
  if (!q || !k_new || !v_new || !k_pool || !v_pool || misaligned16(q, k_new, v_new, k_pool, v_pool)) return ASPD_ERR_INVALID_ARG;
  if (!(p->kernel == ASPD_KERNEL_MMA && p->fuse_append) || attn_mma_direct(p)) return ASPD_ERR_UNSUPPORTED;
  note_stream(p, stream);
  return launch_attn_mma_step(p, q, k_new, v_new, k_pool, v_pool, nullptr, (cudaStream_t)stream);
}

int aspd_attn_combine(aspd_plan_t* p, void* out, void* stream) {
  if (!p || p->host_only) return ASPD_ERR_INVALID_ARG;
  if (p->n_new == 0) return ASPD_OK;
  if (!out || misaligned16(out)) return ASPD_ERR_INVALID_ARG;
  note_stream(p, stream);
  return launch_combine(p, out, (cudaStream_t)stream);
}

static int run_attn(aspd_plan_t* p, int mode, const void* q, const void* k_pool, const void* v_pool, void* out,
                    void* stream) {
  if (!p || p->host_only || p->mode != mode) return ASPD_ERR_INVALID_ARG;
  if (p->n_new == 0) return ASPD_OK;
  if (!q || !k_pool || !v_pool || !out || misaligned16(q, k_pool, v_pool, out)) return ASPD_ERR_INVALID_ARG;
  note_stream(p, stream);
  // a plan with one item per (token, KV head) needs no records: the kernel normalises and writes the output;
  // a single-launch plan's kernel merges its records itself
  if (attn_mma_writes_output(p)) return launch_attn_mma(p, q, k_pool, v_pool, out, (cudaStream_t)stream);
  int rc = aspd_attn_partials(p, q, k_pool, v_pool, stream);
  if (rc) return rc;
  return aspd_attn_combine(p, out, stream);
}

int aspd_branch_attn(aspd_plan_t* p, const void* q, const void* k_pool, const void* v_pool, void* out, void* stream) {
  return run_attn(p, ASPD_MODE_BRANCH, q, k_pool, v_pool, out, stream);
}

int aspd_serial_attn(aspd_plan_t* p, const void* q, const void* k_pool, const void* v_pool, void* out, void* stream) {
  return run_attn(p, ASPD_MODE_SERIAL, q, k_pool, v_pool, out, stream);
}

static int run_step(aspd_plan_t* p, int mode, const void* q, const void* k_new, const void* v_new, void* k_pool,
                    void* v_pool, void* out, void* stream) {
  if (!p || p->host_only || p->mode != mode) return ASPD_ERR_INVALID_ARG;
  if (p->n_new == 0) return ASPD_OK;
  if (!q || !k_new || !v_new || !k_pool || !v_pool || !out || misaligned16(q, k_new, v_new, k_pool, v_pool, out)) return ASPD_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  note_stream(p, stream);
  int rc;
  if (p->kernel == ASPD_KERNEL_MMA && p->fuse_append) {
    rc = launch_attn_mma_step(p, q, k_new, v_new, k_pool, v_pool, out, s);
  } else if (p->kernel == ASPD_KERNEL_MMA) {
    rc = launch_append(p, k_new, v_new, p->dev.tok_pos, k_pool, v_pool, s);
    if (rc == ASPD_OK) rc = launch_attn_mma(p, q, k_pool, v_pool, out, s);
  } else {
    rc = launch_append(p, k_new, v_new, p->dev.tok_pos, k_pool, v_pool, s);
    if (rc == ASPD_OK) rc = launch_attn_generic(p, q, k_pool, v_pool, s);
  }
  if (rc || attn_mma_writes_output(p)) return rc;
  return launch_combine(p, out, s);
}

int aspd_branch_step(aspd_plan_t* p, const void* q, const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                     void* out, void* stream) {
  return run_step(p, ASPD_MODE_BRANCH, q, k_new, v_new, k_pool, v_pool, out, stream);
}

int aspd_serial_step(aspd_plan_t* p, const void* q, const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                     void* out, void* stream) {
  return run_step(p, ASPD_MODE_SERIAL, q, k_new, v_new, k_pool, v_pool, out, stream);
}

int aspd_step_host_async(aspd_plan_t* p, const void* q, const void* k_new, const void* v_new, const int32_t* pos,
                         void* k_pool, void* v_pool, void* out, void* stream) {
  if (!p || p->host_only) return ASPD_ERR_INVALID_ARG;
  if (p->n_new == 0) return ASPD_OK;
  if (!q || !k_new || !v_new || !pos || !k_pool || !v_pool || !out || misaligned16(k_pool, v_pool)) return ASPD_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  note_stream(p, stream);
  const aspd_shape_t& sh = p->shape;
  const size_t es = esize_of(sh.dtype);
  const size_t qb = es * p->n_new * sh.n_q_heads * sh.head_dim, kb = es * p->n_new * sh.n_kv_heads * sh.head_dim;
  // The staging areas of q, k_new and v_new lie back to back in the plan's block; when the caller's
  // three buffers do too (one packed host buffer), one copy moves them all.
  const char* qh = static_cast<const char*>(q);
  const bool packed = static_cast<const char*>(k_new) == qh + qb && static_cast<const char*>(v_new) == qh + qb + kb &&
                      static_cast<char*>(p->dev.st_k) == static_cast<char*>(p->dev.st_q) + qb &&
                      static_cast<char*>(p->dev.st_v) == static_cast<char*>(p->dev.st_q) + qb + kb;
  if (packed) {
    if (cudaMemcpyAsync(p->dev.st_q, q, qb + 2 * kb, cudaMemcpyHostToDevice, s) != cudaSuccess) return ASPD_ERR_CUDA;
  } else if (cudaMemcpyAsync(p->dev.st_q, q, qb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
             cudaMemcpyAsync(p->dev.st_k, k_new, kb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
             cudaMemcpyAsync(p->dev.st_v, v_new, kb, cudaMemcpyHostToDevice, s) != cudaSuccess) {
    return ASPD_ERR_CUDA;
  }
  int rc;
  if (memcmp(pos, p->q_pos.data(), sizeof(int32_t) * p->n_new) == 0) {
    // the caller's position IDs are the plan's (the usual case): they are on the device already,
    // and the step may write the new rows inside the attention pass
    rc = run_step(p, p->mode, p->dev.st_q, p->dev.st_k, p->dev.st_v, k_pool, v_pool, p->dev.st_out, stream);
  } else {
    if (cudaMemcpyAsync(p->dev.st_pos, pos, sizeof(int32_t) * p->n_new, cudaMemcpyHostToDevice, s) != cudaSuccess) return ASPD_ERR_CUDA;
    rc = launch_append(p, p->dev.st_k, p->dev.st_v, p->dev.st_pos, k_pool, v_pool, s);
    if (rc == ASPD_OK) rc = run_attn(p, p->mode, p->dev.st_q, k_pool, v_pool, p->dev.st_out, stream);
  }
  if (rc) return rc;
  if (cudaMemcpyAsync(out, p->dev.st_out, qb, cudaMemcpyDeviceToHost, s) != cudaSuccess) return ASPD_ERR_CUDA;
  return ASPD_OK;
}

int aspd_step_host(aspd_plan_t* p, const void* q, const void* k_new, const void* v_new, const int32_t* pos,
                   void* k_pool, void* v_pool, void* out, void* stream) {
  const int rc = aspd_step_host_async(p, q, k_new, v_new, pos, k_pool, v_pool, out, stream);
  if (rc) return rc;
  if (p->n_new > 0 && cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return ASPD_ERR_CUDA;
  return ASPD_OK;
}

int aspd_k_rerotate(const aspd_shape_t* shape, void* k_pool, const int32_t* pages, const int32_t* rows,
                    const int32_t* delta, int n, void* stream) {
  int rc = check_shape(shape);
  if (rc) return rc;
  if (n < 0) return ASPD_ERR_INVALID_ARG;
  if (n == 0) return ASPD_OK;
  if (!k_pool || !pages || !rows || !delta || misaligned16(k_pool)) return ASPD_ERR_INVALID_ARG;
  return launch_rerotate(shape, k_pool, pages, rows, delta, n, (cudaStream_t)stream);
}

static int check_ranges(const int32_t* ranges, int n_ranges) {
  for (int i = 0; i < n_ranges; ++i) {
    const int32_t* g = ranges + 4 * (size_t)i;
    if (g[0] < 0 || g[1] < 0 || g[2] < 0 || (long)g[1] + g[2] > INT32_MAX) return ASPD_ERR_BAD_DESCRIPTOR;
  }
  return ASPD_OK;
}

int aspd_k_rerotate_ranges(const aspd_shape_t* shape, void* k_pool, const int32_t* page_table, const int32_t* ranges, int n_ranges,
                           void* stream) {
  return aspd_k_rerotate_ranges_layers(shape, &k_pool, 1, page_table, ranges, n_ranges, stream);
}

int aspd_k_rerotate_ranges_layers(const aspd_shape_t* shape, void* const* k_pools, int n_layers, const int32_t* page_table,
                                  const int32_t* ranges, int n_ranges, void* stream) {
  int rc = check_shape(shape);
  if (rc) return rc;
  if (n_ranges < 0 || n_layers < 0) return ASPD_ERR_INVALID_ARG;
  if (n_ranges == 0 || n_layers == 0) return ASPD_OK;
  if (!k_pools || !page_table || !ranges) return ASPD_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (!k_pools[l] || misaligned16(k_pools[l])) return ASPD_ERR_INVALID_ARG;
  if ((rc = check_ranges(ranges, n_ranges))) return rc;
  return launch_rerotate_ranges(shape, k_pools, n_layers, page_table, ranges, n_ranges, (cudaStream_t)stream);
}

int aspd_debug_pool_limit(aspd_plan_t* p, int64_t n_pages) {
  if (!p || p->host_only || n_pages < 0 || n_pages > p->n_pool_pages) return ASPD_ERR_INVALID_ARG;
#ifdef ASPD_DEBUG_BOUNDS
  p->dev.pool_limit = (int32_t)std::min<int64_t>(n_pages, INT32_MAX);
  return ASPD_OK;
#else
  return ASPD_ERR_UNSUPPORTED;
#endif
}

int aspd_debug_profile(void* device_buf, int cta) {
  if (cta < 0) return ASPD_ERR_INVALID_ARG;
  return set_profile_buffer((long long*)device_buf, cta);
}

int aspd_debug_bounded_wait(int64_t limit_cycles, int32_t* status_out, void* stream) {
  if (!status_out || limit_cycles < 0 || limit_cycles > 4000000000LL) return ASPD_ERR_INVALID_ARG;
  int32_t* dev = nullptr;
  if (cudaMalloc(&dev, sizeof(int32_t)) != cudaSuccess) return ASPD_ERR_NOMEM;
  cudaStream_t s = (cudaStream_t)stream;
  int rc = launch_wait_probe(limit_cycles, dev, s);
  if (rc == ASPD_OK && (cudaMemcpyAsync(status_out, dev, sizeof(int32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
                        cudaStreamSynchronize(s) != cudaSuccess))
    rc = ASPD_ERR_CUDA;
  cudaFree(dev);
  return rc;
}

int aspd_debug_read_token(const aspd_shape_t* shape, const void* pool, int64_t page, int row, int kv_head, float* out,
                          void* stream) {
  int rc = check_shape(shape);
  if (rc) return rc;
  if (!pool || !out || page < 0 || row < 0 || row >= shape->page_size || kv_head < 0 || kv_head >= shape->n_kv_heads)
    return ASPD_ERR_INVALID_ARG;
  float* tmp = nullptr;
  if (cudaMalloc(&tmp, sizeof(float) * shape->head_dim) != cudaSuccess) return ASPD_ERR_NOMEM;
  cudaStream_t s = (cudaStream_t)stream;
  rc = launch_read_token(shape, pool, page, row, kv_head, tmp, s);
  if (rc == ASPD_OK && (cudaMemcpyAsync(out, tmp, sizeof(float) * shape->head_dim, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
                        cudaStreamSynchronize(s) != cudaSuccess))
    rc = ASPD_ERR_CUDA;
  cudaFree(tmp);
  return rc;
}

}  // extern "C"
