// Small kernels: RoPE + paged append (a3), the generic CUDA-core attention kernel (any
// supported dtype / head_dim / page_size), the log-sum-exp combine (a7) and a debug reader.
#include "aspd_internal.cuh"
#include "aspd_combine.cuh"

namespace aspd {

namespace {

constexpr float kLog2e = 1.4426950408889634f;

template <typename T> __device__ inline float to_f32(T x);
template <> __device__ inline float to_f32<float>(float x) { return x; }
template <> __device__ inline float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ inline T from_f32(float x);
template <> __device__ inline float from_f32<float>(float x) { return x; }
template <> __device__ inline __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// ------------------------------------------------------------------------------- append
// A thread owns one 16-byte chunk of the first half of a (new token, KV head) row and its partner
// chunk in the second half (the pairs (i, i + d/2)): it rotates that chunk pair of K and copies
// that chunk pair of V.
constexpr int kAppendThreads = 128;
template <typename T>
__global__ void __launch_bounds__(kAppendThreads)
append_kernel(const T* __restrict__ k_new, const T* __restrict__ v_new, const int32_t* __restrict__ pos,
              const int32_t* __restrict__ tok_page, const int32_t* __restrict__ tok_row,
              const double* __restrict__ inv_freq, T* __restrict__ k_pool, T* __restrict__ v_pool,
              int n_new, int n_kv_heads, int head_dim, int page_size, PlanDevice pd) {
  constexpr int VEC = 16 / sizeof(T);
  pdl_launch_dependents();
  const int half = head_dim / 2, chunks = half / VEC;
  const long gid = (long)blockIdx.x * blockDim.x + threadIdx.x;
  const long t = gid / (chunks * n_kv_heads);
  const int h = (int)(gid / chunks % n_kv_heads), c = (int)(gid % chunks);
  double f[VEC];                                   // plan data: may be read before the dependency wait
#pragma unroll
  for (int j = 0; j < VEC; ++j) f[j] = inv_freq[c * VEC + j];
  pdl_wait();
  if (t >= n_new || !bounds_ok(pd, tok_page[t], tok_row[t], page_size)) return;
  // angle reduced to [-pi, pi] in fp64, then fp32 sincos: the error stays near 1e-7 rad
  // however large the position is
  float sn[VEC], cs[VEC];
  const double p = (double)pos[t];
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    double a = p * f[j];
    a -= rint(a * 0.15915494309189535) * 6.283185307179586;
    sincosf((float)a, &sn[j], &cs[j]);
  }
  const uint32_t rb = head_dim * sizeof(T);
  const size_t tb = tile_bytes(page_size, head_dim, sizeof(T));
  const size_t tile0 = (size_t)tok_page[t] * n_kv_heads * tb;
  const int row = tok_row[t];
  const uint32_t o0 = tile_offset(row, c * 16, rb), o1 = tile_offset(row, half * sizeof(T) + c * 16, rb);
  {
    const size_t src = ((size_t)t * n_kv_heads + h) * head_dim;
    uint4 u0 = *reinterpret_cast<const uint4*>(k_new + src + c * VEC);
    uint4 u1 = *reinterpret_cast<const uint4*>(k_new + src + half + c * VEC);
    const uint4 w0 = *reinterpret_cast<const uint4*>(v_new + src + c * VEC);
    const uint4 w1 = *reinterpret_cast<const uint4*>(v_new + src + half + c * VEC);
    T* x0 = reinterpret_cast<T*>(&u0);
    T* x1 = reinterpret_cast<T*>(&u1);
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
      const float a = to_f32(x0[j]), b = to_f32(x1[j]);
      x0[j] = from_f32<T>(a * cs[j] - b * sn[j]);
      x1[j] = from_f32<T>(b * cs[j] + a * sn[j]);
    }
    char* kp = reinterpret_cast<char*>(k_pool) + tile0 + h * tb;
    char* vp = reinterpret_cast<char*>(v_pool) + tile0 + h * tb;
    *reinterpret_cast<uint4*>(kp + o0) = u0;
    *reinterpret_cast<uint4*>(kp + o1) = u1;
    *reinterpret_cast<uint4*>(vp + o0) = w0;
    *reinterpret_cast<uint4*>(vp + o1) = w1;
  }
}

// ------------------------------------------------------------------- cos/sin table of a plan
// q_cs[t][i] = (cos, sin)(pos[t] * inv_freq[i]): the rotation of new token t's query (and, in the
// fused step, of its key).  Same arithmetic as the append kernel: angle reduced in fp64, fp32 sincos.
__global__ void qcs_kernel(const int32_t* __restrict__ pos, const double* __restrict__ inv_freq, float2* __restrict__ q_cs,
                           int n_new, int half) {
  const long gid = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= (long)n_new * half) return;
  const int t = (int)(gid / half), i = (int)(gid % half);
  double a = (double)pos[t] * inv_freq[i];
  a -= rint(a * 0.15915494309189535) * 6.283185307179586;
  float sn, cs;
  sincosf((float)a, &sn, &cs);
  q_cs[gid] = make_float2(cs, sn);
}

// --------------------------------------------------------------------------- re-rotation
// K'(pos + delta) = RoPE(K'(pos), delta): rotations compose, so cached keys can be moved to new
// position IDs in place, reading and writing each key once, instead of being re-encoded from
// the raw keys.  A thread owns one 16-byte chunk of the first half of a token's row and its
// partner chunk in the second half (the pairs (i, i + d/2)), computes the chunk's sines and
// cosines once and applies them to every KV head of the token.
constexpr int kRerotateThreads = 256;
struct InvFreq {          // theta^(-2i/d), computed by the host in double; by value in the launch
  double f[64];
};
// One thread's share of a token: the 16-byte chunk at o0 and its partner at o1 in every KV head's
// tile.  The loads of four heads are issued before the first store (the stores go to the same pool,
// so the compiler would otherwise keep every head's loads behind the previous head's stores).
template <typename T>
__device__ __forceinline__ void rotate_token_heads(char* tile, size_t tb, uint32_t o0, uint32_t o1, int n_kv_heads,
                                                   const float (&sn)[16 / sizeof(T)], const float (&cs)[16 / sizeof(T)]) {
  constexpr int VEC = 16 / sizeof(T);
  for (int h0 = 0; h0 < n_kv_heads; h0 += 4) {
    uint4 u0[4], u1[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int h = min(h0 + k, n_kv_heads - 1);
      u0[k] = *reinterpret_cast<const uint4*>(tile + h * tb + o0);
      u1[k] = *reinterpret_cast<const uint4*>(tile + h * tb + o1);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (h0 + k >= n_kv_heads) break;
      T* x0 = reinterpret_cast<T*>(&u0[k]);
      T* x1 = reinterpret_cast<T*>(&u1[k]);
#pragma unroll
      for (int j = 0; j < VEC; ++j) {
        const float a = to_f32(x0[j]), b = to_f32(x1[j]);
        x0[j] = from_f32<T>(a * cs[j] - b * sn[j]);
        x1[j] = from_f32<T>(b * cs[j] + a * sn[j]);
      }
      *reinterpret_cast<uint4*>(tile + (h0 + k) * tb + o0) = u0[k];
      *reinterpret_cast<uint4*>(tile + (h0 + k) * tb + o1) = u1[k];
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(kRerotateThreads)
rerotate_kernel(T* __restrict__ k_pool, const int32_t* __restrict__ pages, const int32_t* __restrict__ rows,
                const int32_t* __restrict__ delta, const InvFreq table, int n, int n_kv_heads, int head_dim, int page_size) {
  constexpr int VEC = 16 / sizeof(T);
  __shared__ double inv_freq[64];
  pdl_launch_dependents();
  const int half = head_dim / 2, chunks = half / VEC;
  if (threadIdx.x < half) inv_freq[threadIdx.x] = table.f[threadIdx.x];
  __syncthreads();
  pdl_wait();
  const long gid = (long)blockIdx.x * blockDim.x + threadIdx.x;
  const long t = gid / chunks;
  const int c = (int)(gid % chunks);
  if (t >= n) return;
  float sn[VEC], cs[VEC];
  const double dl = (double)delta[t];
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    double a = dl * inv_freq[c * VEC + j];
    a -= rint(a * 0.15915494309189535) * 6.283185307179586;
    sincosf((float)a, &sn[j], &cs[j]);
  }
  const uint32_t rb = head_dim * sizeof(T);
  const size_t tb = tile_bytes(page_size, head_dim, sizeof(T));
  char* tile = reinterpret_cast<char*>(k_pool) + (size_t)pages[t] * n_kv_heads * tb;
  const uint32_t o0 = tile_offset(rows[t], c * 16, rb), o1 = tile_offset(rows[t], half * sizeof(T) + c * 16, rb);
  rotate_token_heads<T>(tile, tb, o0, o1, n_kv_heads, sn, cs);
}

// The same with the tokens given as ranges of logical slots: range i covers `count` consecutive
// slots from `first` of the request whose page table starts at page_table[base], all moved by the
// same `delta` (a finished branch that is renumbered moves as a whole).  The kernel derives page
// and row itself, so no per-token index arrays are read: a block takes one page of one range.
constexpr int kMaxRanges = 512;         // ranges per launch (they travel in the launch parameters, about 10 KB)
struct RerotateRanges {
  int n;
  int unit0[kMaxRanges + 1];            // first page unit of range i (prefix sum of the pages each range touches)
  int4 r[kMaxRanges];                   // (page-table base, first slot, count, delta)
};
constexpr int kMaxLayerPools = 64;      // K pools (layers) per launch: grid.y, their addresses in the launch parameters
struct PoolList {
  void* p[kMaxLayerPools];
};
template <typename T>
__global__ void __launch_bounds__(512)
rerotate_ranges_kernel(const PoolList pools, const int32_t* __restrict__ page_table, const RerotateRanges rr, const InvFreq table,
                       int n_kv_heads, int head_dim, int page_size) {
  T* __restrict__ k_pool = static_cast<T*>(pools.p[blockIdx.y]);   // the layers share the page tables, so the same pages move in each
  constexpr int VEC = 16 / sizeof(T);
  __shared__ float2 cs_sm[64];          // (cos, sin) of the range's delta for every element pair: the same for all tokens of the page
  pdl_launch_dependents();
  const int half = head_dim / 2, chunks = half / VEC;
  const int u = blockIdx.x;
  int lo = 0, hi = rr.n - 1;            // the range this block's page belongs to: last i with unit0[i] <= u
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (rr.unit0[mid] <= u) lo = mid; else hi = mid - 1;
  }
  const int4 rg = rr.r[lo];
  const int page = rg.y / page_size + (u - rr.unit0[lo]);           // index of the page in the request's table
  const int tok = threadIdx.x / chunks, c = threadIdx.x % chunks, slot = page * page_size + tok;
  const bool active = tok < page_size && slot >= rg.y && slot < rg.y + rg.z;
  // the sines and cosines depend on the launch parameters only: taken before the dependency wait,
  // i.e. while the previous kernel of the stream is still running
  if ((int)threadIdx.x < half) {
    double a = (double)rg.w * table.f[threadIdx.x];
    a -= rint(a * 0.15915494309189535) * 6.283185307179586;
    float sn1, cs1;
    sincosf((float)a, &sn1, &cs1);
    cs_sm[threadIdx.x] = make_float2(cs1, sn1);
  }
  __syncthreads();
  pdl_wait();
  const uint32_t rb = head_dim * sizeof(T);
  const size_t tb = tile_bytes(page_size, head_dim, sizeof(T));
  char* tile = reinterpret_cast<char*>(k_pool) + (size_t)page_table[rg.x + page] * n_kv_heads * tb;
  const uint32_t o0 = tile_offset(tok, c * 16, rb), o1 = tile_offset(tok, half * sizeof(T) + c * 16, rb);
  uint4 u0[4], u1[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    u0[k] = make_uint4(0, 0, 0, 0); u1[k] = u0[k];
    if (active) {
      const int h = min(k, n_kv_heads - 1);
      u0[k] = *reinterpret_cast<const uint4*>(tile + h * tb + o0);
      u1[k] = *reinterpret_cast<const uint4*>(tile + h * tb + o1);
    }
  }
  if (!active) return;
  float sn[VEC], cs[VEC];
#pragma unroll
  for (int j = 0; j < VEC; ++j) { cs[j] = cs_sm[c * VEC + j].x; sn[j] = cs_sm[c * VEC + j].y; }
  for (int h0 = 0; h0 < n_kv_heads; h0 += 4) {
    if (h0 > 0) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int h = min(h0 + k, n_kv_heads - 1);
        u0[k] = *reinterpret_cast<const uint4*>(tile + h * tb + o0);
        u1[k] = *reinterpret_cast<const uint4*>(tile + h * tb + o1);
      }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (h0 + k >= n_kv_heads) break;
      T* x0 = reinterpret_cast<T*>(&u0[k]);
      T* x1 = reinterpret_cast<T*>(&u1[k]);
#pragma unroll
      for (int j = 0; j < VEC; ++j) {
        const float a = to_f32(x0[j]), b = to_f32(x1[j]);
        x0[j] = from_f32<T>(a * cs[j] - b * sn[j]);
        x1[j] = from_f32<T>(b * cs[j] + a * sn[j]);
      }
      *reinterpret_cast<uint4*>(tile + (h0 + k) * tb + o0) = u0[k];
      *reinterpret_cast<uint4*>(tile + (h0 + k) * tb + o1) = u1[k];
    }
  }
}

// ------------------------------------------------------------------- generic attention
// One block per work item, one warp per query row at a time.  Lane j scores key j of each
// group of 32 keys (a full dot product against the rotated, pre-scaled query held in shared
// memory); the weighted V sum is taken with each lane owning D/32 output elements.
template <typename T, int D>
__global__ void __launch_bounds__(128) attn_generic_kernel(PlanDevice pd, const T* __restrict__ q,
                                                           const T* __restrict__ k_pool, const T* __restrict__ v_pool,
                                                           int n_q_heads, int n_kv_heads, int page_size, float scale_log2) {
  constexpr int EPL = D / 32;                 // output elements per lane
  constexpr int EPC = 16 / (int)sizeof(T);    // elements per 16-byte chunk
  __shared__ float q_s[4][D];
  pdl_launch_dependents();
  pdl_wait();
  const DeviceItem it = pd.items[blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = n_q_heads / n_kv_heads, n_rows = it.n_q_tok * G, n_keys = it.n_pages * page_size;
  const size_t tb = tile_bytes(page_size, D, sizeof(T));
  for (int r = warp; r < n_rows; r += 4) {
    const int tl = r / G, g = r % G, tok = it.q_tok0 + tl, hq = it.kv_head * G + g;
    // rotate the query at its own position (table built on the host in fp64), fold in the scale
    const T* qrow = q + ((size_t)tok * n_q_heads + hq) * D;
    for (int i = lane; i < D / 2; i += 32) {
      const float2 cs = pd.q_cs[(size_t)tok * (D / 2) + i];
      const float x0 = to_f32(qrow[i]), x1 = to_f32(qrow[i + D / 2]);
      q_s[warp][i] = (x0 * cs.x - x1 * cs.y) * scale_log2;
      q_s[warp][i + D / 2] = (x1 * cs.x + x0 * cs.y) * scale_log2;
    }
    __syncwarp();
    // stream keys [0, pe) and [lo, hi) are visible; under the shared mask (w > 0) also keys of other
    // branches whose offset in their branch (page index in the upper bits of the page entry) is below w
    const int4 vis = pd.tok_vis[tok];
    float m = -INFINITY, l = 0.f, acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    for (int base = 0; base < n_keys; base += 32) {
      const int j = base + lane;
      bool seen = false;
      float s = -INFINITY;
      if (j < n_keys) {
        const int2 pg = pd.visit[it.page0 + j / page_size];
        const int row = j % page_size, kg = it.key0 + j;
        seen = row < (pg.y & 255) && (kg < vis.x || (kg >= vis.y && kg < vis.z) || (pg.y >> 13) * page_size + row < vis.w);
        if (seen && !bounds_ok(pd, pg.x, row, page_size)) seen = false;      // checking builds: flagged, key left out
        if (seen) {
          const char* tile = reinterpret_cast<const char*>(k_pool) + ((size_t)pg.x * n_kv_heads + it.kv_head) * tb;
          float dot = 0.f;
#pragma unroll 4
          for (int c = 0; c < D / EPC; ++c) {
            const uint4 raw = *reinterpret_cast<const uint4*>(tile + tile_offset(row, c * 16, D * sizeof(T)));
            const T* e8 = reinterpret_cast<const T*>(&raw);
#pragma unroll
            for (int e = 0; e < EPC; ++e) dot = fmaf(q_s[warp][c * EPC + e], to_f32(e8[e]), dot);
          }
          s = dot;
        }
      }
      if (!__any_sync(0xffffffffu, seen)) continue;
      float mx = s;
#pragma unroll
      for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m, mx);           // finite: at least one key of the group is seen
      const float p = seen ? exp2f(s - m_new) : 0.f;
      const float alpha = exp2f(m - m_new);       // m = -inf before the first seen key: alpha = 0
      float ps = p;
#pragma unroll
      for (int o = 16; o; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
      l = l * alpha + ps;
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] *= alpha;
      const int cnt = min(32, n_keys - base);
      for (int jj = 0; jj < cnt; ++jj) {
        const float pj = __shfl_sync(0xffffffffu, p, jj);
        if (pj == 0.f) continue;                  // masked (or negligible) key: its V row is not touched
        const int key = base + jj;
        const int2 pg = pd.visit[it.page0 + key / page_size];
        const char* tile = reinterpret_cast<const char*>(v_pool) + ((size_t)pg.x * n_kv_heads + it.kv_head) * tb;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          const T v = *reinterpret_cast<const T*>(tile + tile_offset(key % page_size, (lane * EPL + e) * sizeof(T), D * sizeof(T)));
          acc[e] = fmaf(pj, to_f32(v), acc[e]);
        }
      }
      m = m_new;
    }
    const size_t rec = (size_t)(pd.part_base[tok * n_kv_heads + it.kv_head] + it.part_slot) * G + g;
    if (lane == 0) pd.ws_ml[rec] = make_float2(m, l);
#pragma unroll
    for (int e = 0; e < EPL; ++e) pd.ws_o[rec * D + lane * EPL + e] = acc[e];
    __syncwarp();
  }
}

// ------------------------------------------------------------------------------ combine
// One warp per (new token, query head): merge the partial records of (token, KV head) by
// log-sum-exp in one pass with a running maximum.  Where the records lie is plan data and is
// read before the dependency wait; then each round loads the (max, sum) pairs of eight records
// and their O rows together, so a row with up to eight records costs one memory round trip.
template <typename T, int D>
__global__ void combine_kernel(PlanDevice pd, T* __restrict__ out, int n_new, int n_q_heads, int n_kv_heads) {
  pdl_launch_dependents();
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  const bool active = w < n_new * n_q_heads;
  const int tok = active ? w / n_q_heads : 0, hq = active ? w % n_q_heads : 0;
  const int G = n_q_heads / n_kv_heads, h = hq / G, g = hq % G;
  const int p0 = pd.part_base[tok * n_kv_heads + h], n = pd.part_base[tok * n_kv_heads + h + 1] - p0;
  pdl_wait();
  if (!active) return;
  combine_row<T, D, true>(pd.ws_o, pd.ws_ml, p0, n, G, g, lane, out + ((size_t)tok * n_q_heads + hq) * D);
}

template <typename T>
__global__ void read_token_kernel(const T* pool, size_t tile, int row, int head_dim, float* out) {
  const int e = threadIdx.x;
  out[e] = to_f32(*reinterpret_cast<const T*>(reinterpret_cast<const char*>(pool) + tile + tile_offset(row, e * sizeof(T), head_dim * sizeof(T))));
}

inline int check_launch() { return cudaGetLastError() == cudaSuccess ? ASPD_OK : ASPD_ERR_CUDA; }
inline int status_of(cudaError_t e) { return e == cudaSuccess ? ASPD_OK : ASPD_ERR_CUDA; }

}  // namespace

int launch_append(const aspd_plan* p, const void* k_new, const void* v_new, const int32_t* pos, void* k_pool,
                  void* v_pool, cudaStream_t s) {
  const aspd_shape_t& sh = p->shape;
  const int chunks = sh.head_dim / 2 / (16 / esize_of(sh.dtype));
  const dim3 grid((unsigned)(((long)p->n_new * sh.n_kv_heads * chunks + kAppendThreads - 1) / kAppendThreads)), block(kAppendThreads);
  if (sh.dtype == ASPD_DTYPE_BF16)
    return status_of(launch_pdl(kPdlAppend, append_kernel<__nv_bfloat16>, grid, block, 0, s, (const __nv_bfloat16*)k_new,
                                (const __nv_bfloat16*)v_new, pos, p->dev.tok_page, p->dev.tok_row, p->dev.inv_freq,
                                (__nv_bfloat16*)k_pool, (__nv_bfloat16*)v_pool, p->n_new, sh.n_kv_heads, sh.head_dim, sh.page_size, p->dev));
  return status_of(launch_pdl(kPdlAppend, append_kernel<float>, grid, block, 0, s, (const float*)k_new, (const float*)v_new, pos,
                              p->dev.tok_page, p->dev.tok_row, p->dev.inv_freq, (float*)k_pool, (float*)v_pool, p->n_new,
                              sh.n_kv_heads, sh.head_dim, sh.page_size, p->dev));
}

int launch_attn_generic(const aspd_plan* p, const void* q, const void* k_pool, const void* v_pool, cudaStream_t s) {
  const aspd_shape_t& sh = p->shape;
  if (p->n_items == 0) return ASPD_OK;
  const float sc = sh.sm_scale * kLog2e;
  const dim3 grid(p->n_items), block(128);
#define ASPD_GEN(T, D)                                                                                         \
  return status_of(launch_pdl(kPdlAttn, attn_generic_kernel<T, D>, grid, block, 0, s, p->dev, (const T*)q, (const T*)k_pool, \
                              (const T*)v_pool, sh.n_q_heads, sh.n_kv_heads, sh.page_size, sc))
  if (sh.dtype == ASPD_DTYPE_BF16 && sh.head_dim == 128) ASPD_GEN(__nv_bfloat16, 128);
  else if (sh.dtype == ASPD_DTYPE_BF16) ASPD_GEN(__nv_bfloat16, 64);
  else if (sh.head_dim == 128) ASPD_GEN(float, 128);
  else ASPD_GEN(float, 64);
#undef ASPD_GEN
}

int launch_qcs(const aspd_plan* p, cudaStream_t s) {
  const int half = p->shape.head_dim / 2;
  const long n = (long)p->n_new * half;
  qcs_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(p->dev.tok_pos, p->dev.inv_freq, const_cast<float2*>(p->dev.q_cs), p->n_new, half);
  return check_launch();
}

int launch_combine(const aspd_plan* p, void* out, cudaStream_t s) {
  const aspd_shape_t& sh = p->shape;
  const int warps = p->n_new * sh.n_q_heads;
  const dim3 block(128), grid((warps + 3) / 4);
  // Measured: with the attribute the combine's blocks wait on the SMs while the attention pass
  // ends, which wins a little on a large step (serving mix: 48.6 against 49.2 us per layer) and
  // loses a lot on small ones (long context, one request: 24.9 against 17.6; also with the rows in a
  // few blocks of 32 warps, so that only a few SMs hold combine blocks: 24.7 against 18.2), so it
  // follows the step's size.
  const int which = p->algorithmic_bytes >= (128LL << 20) ? (kPdlCombine | kPdlCombineLarge) : kPdlCombine;
#define ASPD_CMB(T, D) \
  return status_of(launch_pdl(which, combine_kernel<T, D>, grid, block, 0, s, p->dev, (T*)out, p->n_new, sh.n_q_heads, sh.n_kv_heads))
  if (sh.dtype == ASPD_DTYPE_BF16 && sh.head_dim == 128) ASPD_CMB(__nv_bfloat16, 128);
  else if (sh.dtype == ASPD_DTYPE_BF16) ASPD_CMB(__nv_bfloat16, 64);
  else if (sh.head_dim == 128) ASPD_CMB(float, 128);
  else ASPD_CMB(float, 64);
#undef ASPD_CMB
}

int launch_rerotate(const aspd_shape_t* sh, void* k_pool, const int32_t* pages, const int32_t* rows, const int32_t* delta,
                    int n, cudaStream_t s) {
  const int chunks = sh->head_dim / 2 / (16 / esize_of(sh->dtype));
  const dim3 grid((unsigned)(((long)n * chunks + kRerotateThreads - 1) / kRerotateThreads)), block(kRerotateThreads);
  InvFreq table;
  for (int i = 0; i < sh->head_dim / 2; ++i) table.f[i] = pow((double)sh->rope_theta, -2.0 * i / (double)sh->head_dim);
  if (sh->dtype == ASPD_DTYPE_BF16)
    return status_of(launch_pdl(kPdlAppend, rerotate_kernel<__nv_bfloat16>, grid, block, 0, s, (__nv_bfloat16*)k_pool, pages, rows,
                                delta, table, n, sh->n_kv_heads, sh->head_dim, sh->page_size));
  return status_of(launch_pdl(kPdlAppend, rerotate_kernel<float>, grid, block, 0, s, (float*)k_pool, pages, rows, delta,
                              table, n, sh->n_kv_heads, sh->head_dim, sh->page_size));
}

int launch_rerotate_ranges(const aspd_shape_t* sh, void* const* k_pools, int n_layers, const int32_t* page_table,
                           const int32_t* ranges, int n_ranges, cudaStream_t s) {
  const int chunks = sh->head_dim / 2 / (16 / esize_of(sh->dtype)), ps = sh->page_size;
  InvFreq table;
  for (int i = 0; i < sh->head_dim / 2; ++i) table.f[i] = pow((double)sh->rope_theta, -2.0 * i / (double)sh->head_dim);
  for (int r0 = 0; r0 < n_ranges;) {
    RerotateRanges rr;
    rr.n = 0; rr.unit0[0] = 0;
    for (; r0 < n_ranges && rr.n < kMaxRanges; ++r0) {
      const int32_t* g = ranges + 4 * (size_t)r0;
      if (g[2] <= 0) continue;                                   // an empty range moves nothing
      const int pages = (g[1] + g[2] - 1) / ps - g[1] / ps + 1;
      rr.r[rr.n] = make_int4(g[0], g[1], g[2], g[3]);
      rr.unit0[rr.n + 1] = rr.unit0[rr.n] + pages;
      ++rr.n;
    }
    if (rr.n == 0) continue;
    for (int l0 = 0; l0 < n_layers; l0 += kMaxLayerPools) {
      PoolList pools;
      const int nl = std::min(kMaxLayerPools, n_layers - l0);
      for (int l = 0; l < kMaxLayerPools; ++l) pools.p[l] = k_pools[l0 + std::min(l, nl - 1)];
      const dim3 grid((unsigned)rr.unit0[rr.n], (unsigned)nl), block((unsigned)(ps * chunks));
      cudaError_t e;
      if (sh->dtype == ASPD_DTYPE_BF16)
        e = launch_pdl(kPdlAppend, rerotate_ranges_kernel<__nv_bfloat16>, grid, block, 0, s, pools, page_table, rr, table, sh->n_kv_heads,
                       sh->head_dim, ps);
      else
        e = launch_pdl(kPdlAppend, rerotate_ranges_kernel<float>, grid, block, 0, s, pools, page_table, rr, table, sh->n_kv_heads,
                       sh->head_dim, ps);
      if (e != cudaSuccess) return ASPD_ERR_CUDA;
    }
  }
  return ASPD_OK;
}

int launch_read_token(const aspd_shape_t* sh, const void* pool, int64_t page, int row, int kv_head, float* out_dev,
                      cudaStream_t s) {
  const int es = esize_of(sh->dtype);
  const size_t tile = ((size_t)page * sh->n_kv_heads + kv_head) * tile_bytes(sh->page_size, sh->head_dim, es);
  if (sh->dtype == ASPD_DTYPE_BF16)
    read_token_kernel<__nv_bfloat16><<<1, sh->head_dim, 0, s>>>((const __nv_bfloat16*)pool, tile, row, sh->head_dim, out_dev);
  else
    read_token_kernel<float><<<1, sh->head_dim, 0, s>>>((const float*)pool, tile, row, sh->head_dim, out_dev);
  return check_launch();
}

}  // namespace aspd
