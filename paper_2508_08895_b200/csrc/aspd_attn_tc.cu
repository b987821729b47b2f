// Split-K decode attention on the 5th-generation tensor cores (tcgen05 + TMEM), bf16 cache,
// head_dim 128, page_size 16.
//
// One persistent CTA per SM walks its share of the plan's work items.  An item is (query row
// block of one KV head, run of pages of the request's key stream): M = n_q_tok * G <= 64 query rows.
// Keys stream through shared memory in tiles of 128 (8 pages), fetched page by page with
// linear bulk copies (the cache tile format already is the 128-byte-swizzled image the tensor
// core reads).  Per tile:
//
//     S = Qrep . K^T     tcgen05.mma M=128, N=keys, K=128      accumulator in TMEM
//     softmax warps      read S from TMEM, online softmax, write P (bf16) to shared memory
//     O += P . V         tcgen05.mma M=128, N=128, K=keys      accumulator in TMEM
//
// The 128 accumulator lanes are used as R x KS: the query rows (padded to R = 32 or 64) are
// replicated KS = 128 / R times in the A operand, and softmax thread (j, r) handles row r over
// the j-th key sub-range of the tile only, so all 128 threads share the exponentials.  The KS
// threads of a row agree on one reference maximum per tile (exchanged through shared memory)
// and write their P values into the SAME row r of the P tile, so the second MMA sums over all
// keys by itself and rows >= R of its output are simply ignored.  The reference maximum is only
// raised when the tile maximum exceeds it by more than 2^8, which keeps P exactly consistent
// with the (m, l, O) record while making the rescale of O in TMEM rare.
//
// Warp roles: 0-7 softmax (TMEM lane quadrant = warp % 4; warps w and w + 4 share the rows of a
// quadrant and take half of the columns each), 8 and 11 bulk-copy producers (K and V), 9 MMA
// issuer (one elected lane), 12-15 fused append of the step's new rows (aspd_branch_step /
// aspd_serial_step), query preparation (RoPE, bf16, swizzled store, one item ahead) and epilogue
// (TMEM lane quadrant = warp - 12); warp 10 is idle.  All cross-role hand-offs are mbarriers; every
// wait is bounded and on expiry sets the plan's status word to ASPD_ERR_TIMEOUT and makes all
// roles drain and exit.
#include <type_traits>

#include "aspd_internal.cuh"
#include "aspd_combine.cuh"
#include "aspd_tc_common.cuh"

namespace aspd {
namespace {

constexpr int kTile = 128;                     // keys per tile
constexpr int kThreads = 512;
constexpr int kSoftmaxThreads = 256;           // two warps per TMEM lane quadrant, each taking half of the columns
constexpr int W_KPROD = 8, W_MMA = 9, W_VPROD = 11, W_EPI = 12;   // warp roles (0-7 softmax, 10 idle, 12-15 epilogue)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRaise = 8.0f;                 // raise the reference maximum only beyond 2^8
constexpr float kLazyLimit = 1099511627776.0f;  // 2^40: a tile's sum of exponentials beyond which the reference is raised
constexpr float kLower = 32.0f;                // wide variant: lower the initial reference (0) when a row's first keys are below 2^-32

constexpr uint32_t kTileBytes = 32768;         // one K, V, Q or P tile: 128 rows x 256 B
constexpr uint32_t kHalf = 16384;              // second 64-element span of a tile
constexpr uint32_t OFF_K = 0, OFF_V = 2 * kTileBytes, OFF_Q = 4 * kTileBytes, OFF_P = 6 * kTileBytes;
// Rows 64..127 of the P tile are never written (R <= 64) and the rows of O they produce are
// never read, so the barriers and small exchange arrays live in that hole of the first span.
constexpr uint32_t OFF_MISC = OFF_P + 8192;

enum Bar { K_FULL = 0, K_EMPTY = 2, V_FULL = 4, V_EMPTY = 6, S_FULL = 8, S_EMPTY = 10, P_FULL = 12, P_EMPTY = 13,
           O_FULL = 14, O_EMPTY = 16, Q_FULL = 18, Q_EMPTY = 20, E_FULL = 22, A_DONE = 24, NUM_BARS = 25 };

constexpr int kItemCache = 10;      // items of a CTA kept in shared memory (more are read from global)
constexpr int kMergeQueue = 21;     // (token, KV head) pairs whose last record this CTA stored, waiting to be merged
constexpr int kMaxTokPerItem = 16;  // tokens of a row block whose ranges are cached (n_q_tok is at most 64 / G)

// The wide variant of the kernel (row blocks of up to 128 query rows, no replication) fills all
// rows of the P tile; it keeps a single query tile and puts Misc, followed by the reference maxima
// of 2 x 128 rows, where the second query tile would be.
constexpr uint32_t OFF_MISC_WIDE = OFF_Q + kTileBytes;

struct Misc {
  uint64_t bars[NUM_BARS];
  float smax[2][256];          // per S buffer: tile maximum of every softmax thread
  float fin_m[2][64];          // per item parity: reference maximum of every query row ...
  float fin_l[2][256];         // ... and the sum of every softmax thread
  int nval[4][8];              // page entries (valid rows | ... | upper bits) of the 8 pages of a tile (ring over 4 tiles)
  DeviceItem items[kItemCache];        // this CTA's first items and, per item, the visible ranges of
  int4 vis[kItemCache][kMaxTokPerItem]; // its query tokens: no global-load chain at an item boundary
  uint32_t tmem_base;
  int abort_flag;
  int mq_n;                    // merge queue (plans that merge inside the kernel): filled by the epilogue warps with
  int mq[kMergeQueue][3];      // (token * n_kv_heads + KV head, first record, number of records)
};
static_assert(sizeof(Misc) <= 8192, "Misc must fit into the unused rows of the P tile");
constexpr size_t kSmemBytes = 7 * kTileBytes + 1024;   // + slack to align the base to 1024

// TMEM columns: S double buffer, O double buffer
constexpr uint32_t COL_S = 0, COL_O = 256;

#ifdef ASPD_TC_PROFILE
// Development aid (builds with -DASPD_TC_PROFILE): one CTA stamps clock64() at pipeline events of
// its first 64 tiles into the buffer given to aspd_debug_profile.
#define ASPD_STAMP(c, g, ev) do { if ((c).prof && blockIdx.x == (c).prof_cta && (g) < 64) (c).prof[(g) * 16 + (ev)] = clock64(); } while (0)
// every CTA: globaltimer (ns) at entry / after set-up / after its last epilogue / after the final barrier; of the last
// item with records to announce: records stored / fenced / counted; and after the CTA's merges
__device__ __forceinline__ long long gtime() { long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define ASPD_CTA_STAMP(c, ev) do { if ((c).prof) (c).prof[1024 + blockIdx.x * 8 + (ev)] = gtime(); } while (0)
#else
#define ASPD_STAMP(c, g, ev) do { } while (0)
#define ASPD_CTA_STAMP(c, ev) do { } while (0)
#endif

struct Ctx {
  PlanDevice pd;
  long long* prof;
  int prof_cta;
  const __nv_bfloat16* q;
  const __nv_bfloat16* k_new;  // non-null (with v_new): write this step's new rows before reading their pages
  const __nv_bfloat16* v_new;
  const char* k_pool;
  const char* v_pool;
  int n_items, n_q_heads, n_kv_heads;
  float scale_log2;
  int early_fetch;             // plan promise: pages without new rows are not written by in-flight work
  int m64;                     // MMAs with M = 64: row blocks of at most 64 rows are not padded to 128 (half the tensor work)
  int pv64;                    // only P.V with M = 64 (scores and the softmax layout stay at M = 128): O then sits in 16 lanes
                               // of each quadrant (at most 64 of the 128 rows of P.V are ever read)
  int stagger_start;           // plans with few tiles per CTA: the first K tile is requested ahead of the other first tiles
  __nv_bfloat16* out;          // non-null (plans with one item per (token, KV head)): the epilogue writes O / l here
  __nv_bfloat16* merge_out;    // non-null (single-launch plans): the CTA that stores the last record of a (token, KV
                               // head) merges all of them into this; streams with a single item are written directly
};

// Merge the queued (token, KV head) pairs: one warp per (pair, head of the group) at a time, the
// records in slot order (the combine kernel's arithmetic).  Called by `n_warps` warps that have
// passed a barrier after the last push; the caller resets the queue behind another barrier.
__device__ __forceinline__ void drain_merge_queue(const Ctx& c, const Misc* misc, int warp_rank, int n_warps, int lane) {
  const int G = c.n_q_heads / c.n_kv_heads, n = min(misc->mq_n, kMergeQueue) * G;
  for (int u = warp_rank; u < n; u += n_warps) {
    const int idx = misc->mq[u / G][0], g = u % G, tok = idx / c.n_kv_heads, h = idx % c.n_kv_heads;
    const int p0 = misc->mq[u / G][1], np = misc->mq[u / G][2];
    combine_row<__nv_bfloat16, 128>(c.pd.ws_o, c.pd.ws_ml, p0, np, G, g, lane, c.merge_out + ((size_t)tok * c.n_q_heads + h * G + g) * 128);
  }
}

// Item idx of this CTA (rel = idx - item_begin): from the shared-memory cache when it is there.
__device__ __forceinline__ DeviceItem get_item(const Ctx& c, const Misc* misc, int idx, int item_begin) {
  const int rel = idx - item_begin;
  return rel < kItemCache ? misc->items[rel] : c.pd.items[idx];
}

// ------------------------------------------------------------------------------- softmax role
// 16-bit mask with bits [lo, hi) set (arguments are clamped to 0..16).
__device__ __forceinline__ uint32_t bits_between(int lo, int hi) {
  lo = max(lo, 0); hi = min(hi, 16);
  return hi > lo ? ((0xFFFFu >> (16 - hi)) & ~((1u << lo) - 1u)) : 0u;
}

template <int NC>   // NC = padded row count R = columns of a row replica; a thread takes half of them
__device__ __forceinline__ bool softmax_item(const Ctx& c, const DeviceItem& it, Misc* misc, uint32_t bars, uint32_t smem_p,
                                             uint32_t tmem, int item_no, int& g) {   // item_no = index among this CTA's items
  constexpr int R = NC, KS = 128 / NC, HC = NC / 2;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int tl = tid & 127, half = tid >> 7;     // TMEM lane of the thread; which half of the replica's columns
  const int r = tl % R, j = tl / R;
  const int col0 = j * NC + half * HC;           // first tile column (key) of this thread
  const int G = c.n_q_heads / c.n_kv_heads, M = it.n_q_tok * G;
  const int n_tiles = (it.n_pages + 7) >> 3;
  volatile int* ab = &misc->abort_flag;
  int4 vis = make_int4(0, 0, 0, 0);             // padding rows see nothing
  if (r < M) vis = (item_no < kItemCache && r / G < kMaxTokPerItem) ? misc->vis[item_no][r / G] : c.pd.tok_vis[it.q_tok0 + r / G];
  const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
  const bool o_owner = half == 0 && (warp & 3) < R / 32;   // threads whose TMEM lane holds a row of O
  const int ob = item_no & 1;
  float m_ref = -INFINITY, l = 0.f;
  bool dead = false;   // a wait gave up: keep walking the same control flow, report at the end
  for (int t = 0; t < n_tiles; ++t, ++g) {
    const int sb = g & 1;
    dead |= !mbar_wait(bars + 8 * (S_FULL + sb), (g >> 1) & 1, ab);
    tc_fence_after();
    if (tid == 0) ASPD_STAMP(c, g, 0);
    float s[HC];
    const uint32_t s_addr = tmem + lane_addr + COL_S + sb * 128 + col0;
    if constexpr (HC == 32) ASPD_TMEM_LD32(s_addr, s, 0);
    else ASPD_TMEM_LD16(s_addr, s, 0);
    tmem_wait_ld();
    if (tid == 0) ASPD_STAMP(c, g, 1);
    // After an item's first tile the rows have a reference maximum, and a tile's exponentials are
    // taken against it right away: one pass (mask, packed fp32 pairs, the exponentials), no maximum,
    // no exchange between the threads of a row.  The reference then stays where it is unless an
    // exponent passes 2^40, which shows in the sum; the barrier below ORs that over the CTA and the
    // tile is redone the long way (scores read again from TMEM, row maximum exchanged, reference
    // raised, O rescaled).  Everything is floating point, so a reference up to 2^40 below a row's
    // true maximum costs no precision.
    bool lazy = t > 0;
    if (lazy) {
      if (m_ref == -INFINITY) m_ref = 0.f;        // the row has seen nothing so far (l and O are 0): any reference will do
      float2 lsum = make_float2(0.f, 0.f);
      const float2 sc2 = make_float2(c.scale_log2, c.scale_log2), nm2 = make_float2(-m_ref, -m_ref);
#pragma unroll
      for (int pg = 0; pg < HC / 16; ++pg) {
        const int ye = misc->nval[g & 3][col0 / 16 + pg], nv = ye & 255;
        const int kb = it.key0 + t * kTile + col0 + pg * 16;
        const uint32_t mask = bits_between(0, min(nv, vis.x - kb)) | bits_between(vis.y - kb, min(nv, vis.z - kb)) |
                              bits_between(0, min(nv, vis.w - (ye >> 13) * 16));
#pragma unroll
        for (int i = 0; i < 16; i += 2) {
          float2 x = __ffma2_rn(make_float2(s[pg * 16 + i], s[pg * 16 + i + 1]), sc2, nm2);
          if (mask != 0xFFFFu) {
            x.x = (mask >> i) & 1u ? x.x : -INFINITY;
            x.y = (mask >> (i + 1)) & 1u ? x.y : -INFINITY;
          }
          x.x = ex2(x.x); x.y = ex2(x.y);
          s[pg * 16 + i] = x.x; s[pg * 16 + i + 1] = x.y;
          lsum = __fadd2_rn(lsum, x);
        }
      }
      const float tsum = lsum.x + lsum.y;
      lazy = !named_sync_or(1, kSoftmaxThreads, !(tsum <= kLazyLimit));
      if (lazy) {
        l += tsum;
      } else {                                     // rare: the scores again, then the long way
        if constexpr (HC == 32) ASPD_TMEM_LD32(s_addr, s, 0);
        else ASPD_TMEM_LD16(s_addr, s, 0);
        tmem_wait_ld();
      }
    }
    if (tid == 0) ASPD_STAMP(c, g, 2);
    if (!lazy) {
    // visibility of my HC keys: valid rows of each page, and the token's ranges [0, pe), [lo, hi)
    float mx = -INFINITY;
#pragma unroll
    for (int pg = 0; pg < HC / 16; ++pg) {
      const int ye = misc->nval[g & 3][col0 / 16 + pg], nv = ye & 255;
      const int kb = it.key0 + t * kTile + col0 + pg * 16;       // stream key of the page's first row
      // [0, pe), [lo, hi) and, under the shared mask (vis.w > 0), offsets below vis.w in other branches
      const uint32_t mask = bits_between(0, min(nv, vis.x - kb)) | bits_between(vis.y - kb, min(nv, vis.z - kb)) |
                            bits_between(0, min(nv, vis.w - (ye >> 13) * 16));
      if (mask == 0xFFFFu) {
#pragma unroll
        for (int i = 0; i < 16; ++i) mx = fmaxf(mx, s[pg * 16 + i]);
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float v = (mask >> i) & 1u ? s[pg * 16 + i] : -INFINITY;
          s[pg * 16 + i] = v;
          mx = fmaxf(mx, v);
        }
      }
    }
    mx *= c.scale_log2;                           // the scale is positive: max commutes with it
    misc->smax[sb][tid] = mx;
    named_sync(1, kSoftmaxThreads);
    float m_tile = mx;
#pragma unroll
    for (int jj = 0; jj < KS; ++jj)
      m_tile = fmaxf(m_tile, fmaxf(misc->smax[sb][jj * R + r], misc->smax[sb][128 + jj * R + r]));
    const bool upd = m_tile > m_ref + kRaise;     // also true for the first finite maximum (m_ref = -inf)
    float alpha = 1.f;
    if (upd) { alpha = ex2(m_ref - m_tile); m_ref = m_tile; }
    l *= alpha;
    if (t > 0 && c.pv64) {
      // O comes from an M = 64 MMA: row 16 q + i sits in lane i of quadrant q, which is not the lane of
      // the thread that knows the row's factor.  The factors go through shared memory (the other score
      // buffer's exchange array is free), then warps 0..3 rescale their quadrant's 16 rows.
      if (j == 0 && half == 0) misc->smax[sb ^ 1][r] = alpha;
      named_sync(1, kSoftmaxThreads);
      if (half == 0) {
        const int lq = tid & 31, rq = (warp & 3) * 16 + (lq & 15);
        const float a = (lq < 16 && rq < R) ? misc->smax[sb ^ 1][rq] : 1.f;
        if (__any_sync(0xffffffffu, a != 1.f)) {
          dead |= !mbar_wait(bars + 8 * P_EMPTY, (g - 1) & 1, ab);   // PV of the previous tile is done
          tc_fence_after();
          const uint32_t o_addr = tmem + lane_addr + COL_O + ob * 128;
#pragma unroll 1
          for (int q4 = 0; q4 < 4; ++q4) {
            float o[32];
            ASPD_TMEM_LD32(o_addr + q4 * 32, o, 0);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] *= a;
            ASPD_TMEM_ST32(o_addr + q4 * 32, o, 0);
          }
          tmem_wait_st();
          tc_fence_before();
        }
      }
      named_sync(1, kSoftmaxThreads);                // the array is written again in the next long tile
    } else if (t > 0 && o_owner) {                // the owners of rows 0..R-1 rescale O in TMEM
      if (__any_sync(0xffffffffu, upd)) {
        dead |= !mbar_wait(bars + 8 * P_EMPTY, (g - 1) & 1, ab);   // PV of the previous tile is done
        tc_fence_after();
        const uint32_t o_addr = tmem + lane_addr + COL_O + ob * 128;
#pragma unroll 1
        for (int q4 = 0; q4 < 4; ++q4) {
          float o[32];
          ASPD_TMEM_LD32(o_addr + q4 * 32, o, 0);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] *= alpha;
          ASPD_TMEM_ST32(o_addr + q4 * 32, o, 0);
        }
        tmem_wait_st();
        tc_fence_before();
      }
    }
    const float nmsafe = m_ref == -INFINITY ? 0.f : -m_ref;
    float2 lsum = make_float2(0.f, 0.f);
    const float2 sc2 = make_float2(c.scale_log2, c.scale_log2), nm2 = make_float2(nmsafe, nmsafe);
#pragma unroll
    for (int i = 0; i < HC; i += 2) {             // p = 2^(s * scale - m): packed fp32 pairs (one FFMA, one FADD per two scores), two MUFU
      float2 x = __ffma2_rn(make_float2(s[i], s[i + 1]), sc2, nm2);
      x.x = ex2(x.x); x.y = ex2(x.y);
      s[i] = x.x; s[i + 1] = x.y;
      lsum = __fadd2_rn(lsum, x);
    }
    l += lsum.x + lsum.y;
    }
    tc_fence_before();
    mbar_arrive(bars + 8 * (S_EMPTY + sb));       // the scores are not needed again
    if (tid == 0) ASPD_STAMP(c, g, 3);
    if (g > 0) dead |= !mbar_wait(bars + 8 * P_EMPTY, (g - 1) & 1, ab);   // P tile is free again
    if (tid == 0) ASPD_STAMP(c, g, 4);
#pragma unroll
    for (int c8 = 0; c8 < HC / 8; ++c8) {
      const int kk = col0 + c8 * 8;
      const uint32_t addr = smem_p + (kk >> 6) * kHalf + r * 128 + ((((kk & 63) >> 3) ^ (r & 7)) << 4);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pack_bf16(s[c8 * 8 + 0], s[c8 * 8 + 1])),
                   "r"(pack_bf16(s[c8 * 8 + 2], s[c8 * 8 + 3])), "r"(pack_bf16(s[c8 * 8 + 4], s[c8 * 8 + 5])),
                   "r"(pack_bf16(s[c8 * 8 + 6], s[c8 * 8 + 7])) : "memory");
    }
    fence_async_smem();
    tc_fence_before();
    mbar_arrive(bars + 8 * P_FULL);
    if (tid == 0) ASPD_STAMP(c, g, 5);
  }
  // ---- hand the item's statistics to the epilogue warps and move on to the next item
  dead |= !mbar_wait(bars + 8 * (O_EMPTY + ob), ((item_no >> 1) & 1) ^ 1, ab);   // epilogue of item_no - 2 is done
  if (j == 0 && half == 0) misc->fin_m[ob][r] = m_ref;
  misc->fin_l[ob][tid] = l;
  mbar_arrive(bars + 8 * (E_FULL + ob));
  return !named_sync_or(1, kSoftmaxThreads, dead || *ab);
}

// The same role for MMAs with M = 64 (half the tensor work of M = 128 for row blocks of at most 64 rows):
// the 64 accumulator rows hold the R = 32 or 64 padded query rows KS = 64 / R times, and sit in lanes
// 0..15 of each 32-lane quadrant (row 16 q + i in lane i of quadrant q).  A warp reads its quadrant's 16
// lanes with the 16x256b shape, so all 32 threads get data: thread t holds, of every block of 8 columns,
// columns 2 (t % 4), + 1 of rows 16 q + t / 4 and 16 q + t / 4 + 8.  Warps w and w + 4 again take half of a
// replica's key range each, so a thread has as many scores per tile as in the M = 128 layout, now of two
// rows.  P pairs go to shared memory as 4-byte stores (the four threads of a quad fill a 16-byte chunk).
template <int NC>   // NC = padded row count R
__device__ __forceinline__ bool softmax_item_m64(const Ctx& c, const DeviceItem& it, Misc* misc, uint32_t bars, uint32_t smem_p,
                                                 uint32_t tmem, int item_no, int& g) {
  constexpr int R = NC, KS = 64 / NC, NCOL = 128 / KS, NH = NCOL / 2, NB = NH / 8;   // NB blocks of 8 columns per thread and tile
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q = warp & 3, half = warp >> 2, cq = lane & 3, g8 = lane >> 2;
  const int rho_a = 16 * q + g8, rho_b = rho_a + 8;          // accumulator rows of this thread
  const int j = rho_a / R;                                     // their replica (the same for both: R is a multiple of 16)
  const int ra = rho_a % R, rb = rho_b % R;                    // the query rows they stand for
  const int col0 = j * NCOL + half * NH;                       // first tile column (key) of this thread
  const int G = c.n_q_heads / c.n_kv_heads, M = it.n_q_tok * G;
  const int n_tiles = (it.n_pages + 7) >> 3;
  volatile int* ab = &misc->abort_flag;
  int4 vis_a = make_int4(0, 0, 0, 0), vis_b = vis_a;           // padding rows see nothing
  if (ra < M) vis_a = (item_no < kItemCache && ra / G < kMaxTokPerItem) ? misc->vis[item_no][ra / G] : c.pd.tok_vis[it.q_tok0 + ra / G];
  if (rb < M) vis_b = (item_no < kItemCache && rb / G < kMaxTokPerItem) ? misc->vis[item_no][rb / G] : c.pd.tok_vis[it.q_tok0 + rb / G];
  const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
  const bool o_owner = half == 0 && j == 0;                    // threads whose rows are rows of O
  const int ob = item_no & 1;
  float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
  bool dead = false;
  for (int t = 0; t < n_tiles; ++t, ++g) {
    const int sb = g & 1;
    dead |= !mbar_wait(bars + 8 * (S_FULL + sb), (g >> 1) & 1, ab);
    tc_fence_after();
    float s[4 * NB];
    const uint32_t s_addr = tmem + lane_addr + COL_S + sb * 128 + col0;
    if constexpr (NB == 8) ASPD_TMEM_LD16x256_X8(s_addr, s);
    else ASPD_TMEM_LD16x256_X4(s_addr, s);
    tmem_wait_ld();
    // 16-bit masks of the pages this thread's columns lie in, per row
    uint32_t mk_a[NH / 16], mk_b[NH / 16];
#pragma unroll
    for (int pg = 0; pg < NH / 16; ++pg) {
      const int ye = misc->nval[g & 3][col0 / 16 + pg], nv = ye & 255;
      const int kb = it.key0 + t * kTile + col0 + pg * 16;
      const int sh = (ye >> 13) * 16;
      mk_a[pg] = bits_between(0, min(nv, vis_a.x - kb)) | bits_between(vis_a.y - kb, min(nv, vis_a.z - kb)) | bits_between(0, min(nv, vis_a.w - sh));
      mk_b[pg] = bits_between(0, min(nv, vis_b.x - kb)) | bits_between(vis_b.y - kb, min(nv, vis_b.z - kb)) | bits_between(0, min(nv, vis_b.w - sh));
    }
    bool lazy = t > 0;
    if (lazy) {        // one pass against the rows' references (see softmax_item)
      if (m_a == -INFINITY) m_a = 0.f;
      if (m_b == -INFINITY) m_b = 0.f;
      float2 sum_a = make_float2(0.f, 0.f), sum_b = sum_a;
      const float2 sc2 = make_float2(c.scale_log2, c.scale_log2), nm_a = make_float2(-m_a, -m_a), nm_b = make_float2(-m_b, -m_b);
#pragma unroll
      for (int n = 0; n < NB; ++n) {
        const int bit = (n & 1) * 8 + 2 * cq;
        float2 xa = __ffma2_rn(make_float2(s[4 * n], s[4 * n + 1]), sc2, nm_a);
        float2 xb = __ffma2_rn(make_float2(s[4 * n + 2], s[4 * n + 3]), sc2, nm_b);
        const uint32_t ma = mk_a[n >> 1] >> bit, mb = mk_b[n >> 1] >> bit;
        if ((ma & 3u) != 3u) { xa.x = ma & 1u ? xa.x : -INFINITY; xa.y = ma & 2u ? xa.y : -INFINITY; }
        if ((mb & 3u) != 3u) { xb.x = mb & 1u ? xb.x : -INFINITY; xb.y = mb & 2u ? xb.y : -INFINITY; }
        xa.x = ex2(xa.x); xa.y = ex2(xa.y); xb.x = ex2(xb.x); xb.y = ex2(xb.y);
        s[4 * n] = xa.x; s[4 * n + 1] = xa.y; s[4 * n + 2] = xb.x; s[4 * n + 3] = xb.y;
        sum_a = __fadd2_rn(sum_a, xa);
        sum_b = __fadd2_rn(sum_b, xb);
      }
      const float ta = sum_a.x + sum_a.y, tb = sum_b.x + sum_b.y;
      lazy = !named_sync_or(1, kSoftmaxThreads, !(ta <= kLazyLimit) || !(tb <= kLazyLimit));
      if (lazy) {
        l_a += ta; l_b += tb;
      } else {                                     // rare: the scores again, then the long way
        if constexpr (NB == 8) ASPD_TMEM_LD16x256_X8(s_addr, s);
        else ASPD_TMEM_LD16x256_X4(s_addr, s);
        tmem_wait_ld();
      }
    }
    if (!lazy) {
      float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
      for (int n = 0; n < NB; ++n) {
        const int bit = (n & 1) * 8 + 2 * cq;
        const uint32_t ma = mk_a[n >> 1] >> bit, mb = mk_b[n >> 1] >> bit;
        s[4 * n] = ma & 1u ? s[4 * n] : -INFINITY;         s[4 * n + 1] = ma & 2u ? s[4 * n + 1] : -INFINITY;
        s[4 * n + 2] = mb & 1u ? s[4 * n + 2] : -INFINITY; s[4 * n + 3] = mb & 2u ? s[4 * n + 3] : -INFINITY;
        mx_a = fmaxf(mx_a, fmaxf(s[4 * n], s[4 * n + 1]));
        mx_b = fmaxf(mx_b, fmaxf(s[4 * n + 2], s[4 * n + 3]));
      }
      // row maxima: over the quad, then (through shared memory) over the two halves and the replicas
#pragma unroll
      for (int o = 1; o <= 2; o <<= 1) {
        mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, o));
        mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, o));
      }
      mx_a *= c.scale_log2; mx_b *= c.scale_log2;          // the scale is positive: max commutes with it
      if (cq == 0) { misc->smax[sb][half * 64 + rho_a] = mx_a; misc->smax[sb][half * 64 + rho_b] = mx_b; }
      named_sync(1, kSoftmaxThreads);
      float t_a = -INFINITY, t_b = -INFINITY;
#pragma unroll
      for (int jj = 0; jj < KS; ++jj) {
        t_a = fmaxf(t_a, fmaxf(misc->smax[sb][jj * R + ra], misc->smax[sb][64 + jj * R + ra]));
        t_b = fmaxf(t_b, fmaxf(misc->smax[sb][jj * R + rb], misc->smax[sb][64 + jj * R + rb]));
      }
      const bool upd_a = t_a > m_a + kRaise, upd_b = t_b > m_b + kRaise;   // also the first finite maximum (m = -inf)
      float al_a = 1.f, al_b = 1.f;
      if (upd_a) { al_a = ex2(m_a - t_a); m_a = t_a; }
      if (upd_b) { al_b = ex2(m_b - t_b); m_b = t_b; }
      l_a *= al_a; l_b *= al_b;
      if (t > 0 && o_owner) {                       // the owners of rows 0..R-1 rescale O in TMEM (warp-wide)
        if (__any_sync(0xffffffffu, upd_a || upd_b)) {
          dead |= !mbar_wait(bars + 8 * P_EMPTY, (g - 1) & 1, ab);   // PV of the previous tile is done
          tc_fence_after();
          const uint32_t o_addr = tmem + lane_addr + COL_O + ob * 128;
#pragma unroll 1
          for (int q4 = 0; q4 < 4; ++q4) {
            float o[16];
            ASPD_TMEM_LD16x256_X4(o_addr + q4 * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int n = 0; n < 4; ++n) { o[4 * n] *= al_a; o[4 * n + 1] *= al_a; o[4 * n + 2] *= al_b; o[4 * n + 3] *= al_b; }
            ASPD_TMEM_ST16x256_X4(o_addr + q4 * 32, o);
          }
          tmem_wait_st();
          tc_fence_before();
        }
      }
      const float na = m_a == -INFINITY ? 0.f : -m_a, nb = m_b == -INFINITY ? 0.f : -m_b;
      float2 sum_a = make_float2(0.f, 0.f), sum_b = sum_a;
      const float2 sc2 = make_float2(c.scale_log2, c.scale_log2), nm_a = make_float2(na, na), nm_b = make_float2(nb, nb);
#pragma unroll
      for (int n = 0; n < NB; ++n) {
        float2 xa = __ffma2_rn(make_float2(s[4 * n], s[4 * n + 1]), sc2, nm_a);
        float2 xb = __ffma2_rn(make_float2(s[4 * n + 2], s[4 * n + 3]), sc2, nm_b);
        xa.x = ex2(xa.x); xa.y = ex2(xa.y); xb.x = ex2(xb.x); xb.y = ex2(xb.y);
        s[4 * n] = xa.x; s[4 * n + 1] = xa.y; s[4 * n + 2] = xb.x; s[4 * n + 3] = xb.y;
        sum_a = __fadd2_rn(sum_a, xa);
        sum_b = __fadd2_rn(sum_b, xb);
      }
      l_a += sum_a.x + sum_a.y; l_b += sum_b.x + sum_b.y;
    }
    tc_fence_before();
    mbar_arrive(bars + 8 * (S_EMPTY + sb));       // the scores are not needed again
    if (g > 0) dead |= !mbar_wait(bars + 8 * P_EMPTY, (g - 1) & 1, ab);   // P tile is free again
#pragma unroll
    for (int n = 0; n < NB; ++n) {
      const int kk = col0 + 8 * n;                 // first key of the 16-byte chunk the quad fills
      const uint32_t ch = (uint32_t)(kk >> 6) * kHalf + 4u * cq;
      const uint32_t addr_a = smem_p + ch + ra * 128 + ((((kk & 63) >> 3) ^ (ra & 7)) << 4);
      const uint32_t addr_b = smem_p + ch + rb * 128 + ((((kk & 63) >> 3) ^ (rb & 7)) << 4);
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr_a), "r"(pack_bf16(s[4 * n], s[4 * n + 1])) : "memory");
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr_b), "r"(pack_bf16(s[4 * n + 2], s[4 * n + 3])) : "memory");
    }
    fence_async_smem();
    tc_fence_before();
    mbar_arrive(bars + 8 * P_FULL);
  }
  // ---- hand the item's statistics to the epilogue warps and move on to the next item
  dead |= !mbar_wait(bars + 8 * (O_EMPTY + ob), ((item_no >> 1) & 1) ^ 1, ab);   // epilogue of item_no - 2 is done
#pragma unroll
  for (int o = 1; o <= 2; o <<= 1) {               // the quad's share of the rows' sums
    l_a += __shfl_xor_sync(0xffffffffu, l_a, o);
    l_b += __shfl_xor_sync(0xffffffffu, l_b, o);
  }
  if (cq == 0) {
    if (o_owner) { misc->fin_m[ob][ra] = m_a; misc->fin_m[ob][rb] = m_b; }
    misc->fin_l[ob][half * 128 + j * R + ra] = l_a;
    misc->fin_l[ob][half * 128 + j * R + rb] = l_b;
  }
  mbar_arrive(bars + 8 * (E_FULL + ob));
  return !named_sync_or(1, kSoftmaxThreads, dead || *ab);
}

// Row blocks of 65..128 query rows: every TMEM lane is a row of its own (no replication), thread
// (half, r) takes columns [64 half, 64 half + 64) of row r in two chunks of 32.  One pass per
// tile: the exponentials are taken against the current reference maximum while the largest
// exponent is tracked; only when a row's largest exponent exceeds 2^8 (always on the row's first
// visible key) the reference is raised and the warp repeats the pass from TMEM.
__device__ __forceinline__ bool softmax_item_wide(const Ctx& c, const DeviceItem& it, Misc* misc, uint32_t bars, uint32_t smem_p,
                                                  uint32_t tmem, int item_no, int& g) {
  const int tid = threadIdx.x, warp = tid >> 5;
  const int r = tid & 127, half = tid >> 7;
  const int col0 = half * 64;
  const int G = c.n_q_heads / c.n_kv_heads, M = it.n_q_tok * G;
  const int n_tiles = (it.n_pages + 7) >> 3;
  volatile int* ab = &misc->abort_flag;
  float* fin_m_wide = reinterpret_cast<float*>(misc + 1);
  int4 vis = make_int4(0, 0, 0, 0);
  if (r < M) vis = (item_no < kItemCache && r / G < kMaxTokPerItem) ? misc->vis[item_no][r / G] : c.pd.tok_vis[it.q_tok0 + r / G];
  const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
  const bool o_owner = half == 0;
  const int ob = item_no & 1;
  // The reference starts at 0 (exponents of typical logits are within +-2^8 of it, so the first
  // tile needs no second pass); until the row has seen a key it may also be lowered.
  float m_ref = 0.f, l = 0.f;
  bool seen = false;
  bool dead = false;
  for (int t = 0; t < n_tiles; ++t, ++g) {
    const int sb = g & 1;
    dead |= !mbar_wait(bars + 8 * (S_FULL + sb), (g >> 1) & 1, ab);
    tc_fence_after();
    if (tid == 0) ASPD_STAMP(c, g, 0);
    const uint32_t s_addr = tmem + lane_addr + COL_S + sb * 128 + col0;
    uint32_t pk[32];                                // the row's 64 probabilities of this tile, bf16 pairs
    float tile_sum, tmax;
    // p = 2^(s * scale - base) for the thread's 64 columns; tmax = largest exponent
    auto pass = [&](float base) {
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
      float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
      const float nb = -base;
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        float s[32];
        ASPD_TMEM_LD32(s_addr + ch * 32, s, 0);
        tmem_wait_ld();
#pragma unroll
        for (int pg = 0; pg < 2; ++pg) {
          const int ye = misc->nval[g & 3][col0 / 16 + ch * 2 + pg], nv = ye & 255;
          const int kb = it.key0 + t * kTile + col0 + ch * 32 + pg * 16;
          const uint32_t mask = bits_between(0, min(nv, vis.x - kb)) | bits_between(vis.y - kb, min(nv, vis.z - kb)) |
                                bits_between(0, min(nv, vis.w - (ye >> 13) * 16));
#pragma unroll
          for (int i = 0; i < 16; i += 4) {
            float e0 = fmaf(s[pg * 16 + i], c.scale_log2, nb), e1 = fmaf(s[pg * 16 + i + 1], c.scale_log2, nb);
            float e2 = fmaf(s[pg * 16 + i + 2], c.scale_log2, nb), e3 = fmaf(s[pg * 16 + i + 3], c.scale_log2, nb);
            if (mask != 0xFFFFu) {
              e0 = (mask >> i) & 1u ? e0 : -INFINITY;
              e1 = (mask >> (i + 1)) & 1u ? e1 : -INFINITY;
              e2 = (mask >> (i + 2)) & 1u ? e2 : -INFINITY;
              e3 = (mask >> (i + 3)) & 1u ? e3 : -INFINITY;
            }
            mx0 = fmaxf(mx0, e0); mx1 = fmaxf(mx1, e1); mx2 = fmaxf(mx2, e2); mx3 = fmaxf(mx3, e3);
            e0 = ex2(e0); e1 = ex2(e1); e2 = ex2(e2); e3 = ex2(e3);
            sum0 += e0; sum1 += e1; sum2 += e2; sum3 += e3;
            pk[ch * 16 + pg * 8 + (i >> 1)] = pack_bf16(e0, e1);
            pk[ch * 16 + pg * 8 + (i >> 1) + 1] = pack_bf16(e2, e3);
          }
        }
      }
      tile_sum = (sum0 + sum1) + (sum2 + sum3);
      tmax = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
    };
    pass(m_ref);
    if (tid == 0) ASPD_STAMP(c, g, 1);
    misc->smax[sb][tid] = tmax;
    named_sync(1, kSoftmaxThreads);
    if (tid == 0) ASPD_STAMP(c, g, 2);
    const float row_tmax = fmaxf(misc->smax[sb][r], misc->smax[sb][128 + r]);
    // move the reference: up when an exponent passed 2^8; down only while the row has not seen a
    // key yet (l and its row of O are still exactly 0, so nothing is rescaled then)
    const bool raise = row_tmax > kRaise, lower = !seen && row_tmax < -kLower && row_tmax > -INFINITY;
    const bool upd = raise || lower;
    seen |= row_tmax > -INFINITY;
    float alpha = 1.f;
    if (raise) alpha = ex2(-row_tmax);
    if (upd) m_ref += row_tmax;
    l *= alpha;
    const bool any_upd = __any_sync(0xffffffffu, upd);
    if (t > 0 && o_owner && any_upd) {              // the owners of the rows rescale O in TMEM
      dead |= !mbar_wait(bars + 8 * P_EMPTY, (g - 1) & 1, ab);   // PV of the previous tile is done
      tc_fence_after();
      const uint32_t o_addr = tmem + lane_addr + COL_O + ob * 128;
#pragma unroll 1
      for (int q4 = 0; q4 < 4; ++q4) {
        float o[32];
        ASPD_TMEM_LD32(o_addr + q4 * 32, o, 0);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] *= alpha;
        ASPD_TMEM_ST32(o_addr + q4 * 32, o, 0);
      }
      tmem_wait_st();
    }
    if (any_upd) pass(m_ref);   // the whole warp again (TMEM loads are warp-wide)
    l += tile_sum;
    tc_fence_before();
    mbar_arrive(bars + 8 * (S_EMPTY + sb));
    if (tid == 0) ASPD_STAMP(c, g, 3);
    if (g > 0) dead |= !mbar_wait(bars + 8 * P_EMPTY, (g - 1) & 1, ab);
    if (tid == 0) ASPD_STAMP(c, g, 4);
#pragma unroll
    for (int c8 = 0; c8 < 8; ++c8) {
      const int kk = col0 + c8 * 8;
      const uint32_t addr = smem_p + (kk >> 6) * kHalf + r * 128 + ((((kk & 63) >> 3) ^ (r & 7)) << 4);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pk[c8 * 4 + 0]), "r"(pk[c8 * 4 + 1]),
                   "r"(pk[c8 * 4 + 2]), "r"(pk[c8 * 4 + 3]) : "memory");
    }
    fence_async_smem();
    tc_fence_before();
    mbar_arrive(bars + 8 * P_FULL);
    if (tid == 0) ASPD_STAMP(c, g, 5);
  }
  dead |= !mbar_wait(bars + 8 * (O_EMPTY + ob), ((item_no >> 1) & 1) ^ 1, ab);
  if (half == 0) fin_m_wide[ob * 128 + r] = m_ref;
  misc->fin_l[ob][tid] = l;
  mbar_arrive(bars + 8 * (E_FULL + ob));
  return !named_sync_or(1, kSoftmaxThreads, dead || *ab);
}

// Rotate the item's query rows (RoPE at the token's position, cos/sin table from the plan),
// round to bf16 and store them, replicated KS = 128 / R times, as the 128-byte-swizzled K-major
// A operand.  Called by the 128 epilogue threads (rank 0..127); all loads of a thread's rows
// are issued before the first use.  Unit e = (row e / 8, 16-byte chunk e % 8 of each span); a
// call covers units e0 + rank + 128 u, u < 4 (row blocks of 128 rows need two calls).
struct QUnits {
  uint32_t lo[4][4], hi[4][4];   // per unit: the rotated chunk of the first and of the second span, bf16 pairs
};
// tile128: the rows always form a 128-row tile of their own (no replication), however few they are
__device__ __forceinline__ void prep_q_compute(const Ctx& c, const DeviceItem& it, int rank, int e0, QUnits& qu, bool tile128 = false) {
  const int G = c.n_q_heads / c.n_kv_heads;
  const int M = it.n_q_tok * G, R = tile128 ? 128 : (M <= 32 ? 32 : (M <= 64 ? 64 : 128));
  uint4 a[4], b[4];
  float4 w[4][4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int e = e0 + rank + u * 128, r = e >> 3, ch = e & 7;
    a[u] = make_uint4(0, 0, 0, 0); b[u] = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int i = 0; i < 4; ++i) w[u][i] = make_float4(1.f, 0.f, 1.f, 0.f);
    if (e < R * 8 && r < M) {
      const int tok = it.q_tok0 + r / G, hq = it.kv_head * G + r % G;
      const __nv_bfloat16* qrow = c.q + ((size_t)tok * c.n_q_heads + hq) * 128;
      a[u] = *reinterpret_cast<const uint4*>(qrow + ch * 8);
      b[u] = *reinterpret_cast<const uint4*>(qrow + 64 + ch * 8);
      const float4* cs = reinterpret_cast<const float4*>(c.pd.q_cs + (size_t)tok * 64 + ch * 8);
#pragma unroll
      for (int i = 0; i < 4; ++i) w[u][i] = cs[i];              // (cos, sin) of elements 2i and 2i+1 of the chunk
    }
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const __nv_bfloat162* a2 = reinterpret_cast<const __nv_bfloat162*>(&a[u]);
    const __nv_bfloat162* b2 = reinterpret_cast<const __nv_bfloat162*>(&b[u]);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 x0 = __bfloat1622float2(a2[i]), x1 = __bfloat1622float2(b2[i]);
      qu.lo[u][i] = pack_bf16(x0.x * w[u][i].x - x1.x * w[u][i].y, x0.y * w[u][i].z - x1.y * w[u][i].w);
      qu.hi[u][i] = pack_bf16(x1.x * w[u][i].x + x0.x * w[u][i].y, x1.y * w[u][i].z + x0.y * w[u][i].w);
    }
  }
}
__device__ __forceinline__ void prep_q_store(const Ctx& c, const DeviceItem& it, uint32_t qbuf, int rank, int e0, const QUnits& qu,
                                             bool tile128 = false) {
  const int G = c.n_q_heads / c.n_kv_heads;
  const int M = it.n_q_tok * G, R = tile128 ? 128 : (M <= 32 ? 32 : (M <= 64 ? 64 : 128)), KS = (c.m64 && !tile128 ? 64 : 128) / R;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int e = e0 + rank + u * 128, r = e >> 3, ch = e & 7;
    if (e >= R * 8) break;
    for (int jj = 0; jj < KS; ++jj) {
      const uint32_t addr = qbuf + (jj * R + r) * 128 + ((ch ^ (r & 7)) << 4);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(qu.lo[u][0]), "r"(qu.lo[u][1]), "r"(qu.lo[u][2]),
                   "r"(qu.lo[u][3]) : "memory");
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr + kHalf), "r"(qu.hi[u][0]), "r"(qu.hi[u][1]), "r"(qu.hi[u][2]),
                   "r"(qu.hi[u][3]) : "memory");
    }
  }
}
__device__ __forceinline__ void prep_q(const Ctx& c, const DeviceItem& it, uint32_t qbuf, int rank, int e0 = 0) {
  QUnits qu;
  prep_q_compute(c, it, rank, e0, qu);
  prep_q_store(c, it, qbuf, rank, e0, qu);
}

// Fused step (aspd_branch_step / aspd_serial_step): the rows this step adds to pages that THIS CTA
// reads are written into the pools at the start of the kernel, K rotated at the token's position
// (cos/sin table of the plan) and V as is.  CTAs that read the same page write identical bytes, so
// no cross-CTA ordering is needed.  One unit = one 16-byte chunk pair of K (8 per row) or one
// 16-byte chunk of V (16 per row).  Called by the 128 epilogue threads; the loads of a batch of
// units are all issued before its first store.
__device__ __forceinline__ void append_new_rows(const Ctx& c, int rank, int d0, int n_units, const int4 (&first)[2]) {
  for (int u0 = rank; u0 < n_units; u0 += 128 * 2) {
    int4 d[2];
    uint4 a[2], b[2];
    float4 w[2][4];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int u = u0 + k * 128;
      d[k] = first[k];                                         // the first batch was fetched during set-up
      if (u0 != rank) { d[k] = make_int4(0, 0, 0, 0); if (u < n_units) d[k] = c.pd.dirty[d0 + u / 24]; }   // (page, KV head, token, row)
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int u = u0 + k * 128, sub = u % 24;
      a[k] = make_uint4(0, 0, 0, 0); b[k] = a[k];
      if (u >= n_units) continue;
      const size_t src = ((size_t)d[k].z * c.n_kv_heads + d[k].y) * 128;
      if (sub < 8) {
        a[k] = *reinterpret_cast<const uint4*>(c.k_new + src + sub * 8);
        b[k] = *reinterpret_cast<const uint4*>(c.k_new + src + 64 + sub * 8);
        const float4* cs = reinterpret_cast<const float4*>(c.pd.q_cs + (size_t)d[k].z * 64 + sub * 8);
#pragma unroll
        for (int i = 0; i < 4; ++i) w[k][i] = cs[i];
      } else {
        a[k] = *reinterpret_cast<const uint4*>(c.v_new + src + (sub - 8) * 8);
      }
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int u = u0 + k * 128, sub = u % 24;
      if (u >= n_units || !bounds_ok(c.pd, d[k].x, d[k].w, 16)) continue;
      const size_t tile = ((size_t)d[k].x * c.n_kv_heads + d[k].y) * 4096;
      if (sub < 8) {
        const __nv_bfloat162* a2 = reinterpret_cast<const __nv_bfloat162*>(&a[k]);
        const __nv_bfloat162* b2 = reinterpret_cast<const __nv_bfloat162*>(&b[k]);
        uint32_t lo[4], hi[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 x0 = __bfloat1622float2(a2[i]), x1 = __bfloat1622float2(b2[i]);
          lo[i] = pack_bf16(x0.x * w[k][i].x - x1.x * w[k][i].y, x0.y * w[k][i].z - x1.y * w[k][i].w);
          hi[i] = pack_bf16(x1.x * w[k][i].x + x0.x * w[k][i].y, x1.y * w[k][i].z + x0.y * w[k][i].w);
        }
        char* kt = const_cast<char*>(c.k_pool) + tile;
        *reinterpret_cast<uint4*>(kt + tile_offset(d[k].w, sub * 16, 256)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        *reinterpret_cast<uint4*>(kt + tile_offset(d[k].w, 128 + sub * 16, 256)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      } else {
        *reinterpret_cast<uint4*>(const_cast<char*>(c.v_pool) + tile + tile_offset(d[k].w, (sub - 8) * 16, 256)) = a[k];
      }
    }
  }
  asm volatile("fence.proxy.async;" ::: "memory");   // generic-proxy stores before the producers' async-proxy copies
}

// --------------------------------------------------------------------------------- the kernel
// WIDE: row blocks of up to 128 query rows (plans that deal whole streams to the CTAs); one
// query tile instead of two, Misc in the place of the second.
template <bool WIDE>
__global__ void __launch_bounds__(kThreads, 1) attn_tc_kernel(Ctx c) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  constexpr uint32_t off_misc = WIDE ? OFF_MISC_WIDE : OFF_MISC;
  Misc* misc = reinterpret_cast<Misc*>(smem + off_misc);
  const uint32_t bars = base + off_misc;          // bars[] is the first member of Misc
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* ab = &misc->abort_flag;
  if (tid == 0) ASPD_CTA_STAMP(c, 0);
  if (tid == 0) pdl_launch_dependents();
  const int4 head = c.pd.cta_head[blockIdx.x];
  const int item_begin = head.x, item_end = head.y;
  // Plan tables do not depend on earlier kernels of the stream: the CTA's items and, for the
  // producers, the first batch of page entries (whose place comes with the head entry, so that it
  // is the second load of the kernel, not the fourth) are fetched while the CTA is still setting up.
  int2 first_pages = make_int2(0, 0);
  if ((warp == W_KPROD || warp == W_VPROD) && lane < head.w) first_pages = c.pd.visit[head.z + lane];
  {
    const int n_cached = min(item_end - item_begin, kItemCache);
    for (int e = tid; e < n_cached * (int)(sizeof(DeviceItem) / 4); e += kThreads)
      reinterpret_cast<int*>(misc->items)[e] = reinterpret_cast<const int*>(c.pd.items + item_begin)[e];
    for (int e = tid; e < n_cached * kMaxTokPerItem; e += kThreads) {
      const DeviceItem& ci = c.pd.items[item_begin + e / kMaxTokPerItem];
      const int tl = e % kMaxTokPerItem;
      if (tl < ci.n_q_tok) misc->vis[e / kMaxTokPerItem][tl] = c.pd.tok_vis[ci.q_tok0 + tl];
    }
  }

  if (tid == 0) {
    const int counts[NUM_BARS] = {1, 1, 1, 1, 1, 1, 1, 1, 1, 1, 256, 256, 256, 1, 1, 1, 128, 128, 128, 128, 1, 1, 256, 256, 128};
    for (int i = 0; i < NUM_BARS; ++i) mbar_init(bars + 8 * i, counts[i]);
    misc->abort_flag = 0;
    misc->mq_n = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&misc->tmem_base)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc->tmem_base;
  // fused step: the epilogue threads fetch their first new-row entries now (plan data)
  int dirty0 = 0, dirty_units = 0;
  int4 dirty_first[2] = {make_int4(0, 0, 0, 0), make_int4(0, 0, 0, 0)};
  if (warp >= W_EPI && c.k_new != nullptr) {
    dirty0 = c.pd.cta_dirty0[blockIdx.x];
    dirty_units = (c.pd.cta_dirty0[blockIdx.x + 1] - dirty0) * 24;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int u = (tid - W_EPI * 32) + k * 128;
      if (u < dirty_units) dirty_first[k] = c.pd.dirty[dirty0 + u / 24];
    }
  }
  // everything above touches only the plan's own tables; inputs written by earlier kernels of
  // the stream (q, k_new, the pools, the workspace's previous readers) are used from here on.
  // With the plan's stable-cache promise the two producer warps go ahead and fetch pages that
  // hold no new rows; they wait themselves before the first page that does.
  const bool producer_runs_ahead = c.early_fetch && (warp == W_KPROD || warp == W_VPROD);
  if (!producer_runs_ahead) pdl_wait();
  if (tid == 0) ASPD_CTA_STAMP(c, 1);

  if (warp < 8) {
    // =============================== softmax ===============================
    int g = 0, item_no = 0;
    for (int idx = item_begin; idx < item_end; ++idx, ++item_no) {
      const DeviceItem it = get_item(c, misc, idx, item_begin);
      const int M = it.n_q_tok * (c.n_q_heads / c.n_kv_heads);
      bool ok;
      if constexpr (WIDE) {
        ok = M <= 32 ? softmax_item<32>(c, it, misc, bars, base + OFF_P, tmem, item_no, g)
           : M <= 64 ? softmax_item<64>(c, it, misc, bars, base + OFF_P, tmem, item_no, g)
                     : softmax_item_wide(c, it, misc, bars, base + OFF_P, tmem, item_no, g);
      } else {
        if (c.m64)
          ok = M <= 32 ? softmax_item_m64<32>(c, it, misc, bars, base + OFF_P, tmem, item_no, g)
                       : softmax_item_m64<64>(c, it, misc, bars, base + OFF_P, tmem, item_no, g);
        else
          ok = M <= 32 ? softmax_item<32>(c, it, misc, bars, base + OFF_P, tmem, item_no, g)
                       : softmax_item<64>(c, it, misc, bars, base + OFF_P, tmem, item_no, g);
      }
      if (!ok) break;
    }
  } else if (warp == W_KPROD || warp == W_VPROD) {
    // ================================ bulk-copy producers ================================
    // Warp 8 streams the K tiles and warp 11 the V tiles, each on its own ring, so that a K load
    // never queues behind a V slot that is still being read (and vice versa).
    // Lane l keeps stream-page entry (batch * 32 + l) of the item in a register; the next batch
    // of 32 entries (4 tiles) is requested before the current one is consumed, so the page list
    // never sits on the critical path.
    const int kv = warp == W_KPROD ? 0 : 1;
    const char* pool = kv ? c.v_pool : c.k_pool;
    int g = 0;
    bool ok = true, appended = false, waited = false;
    // (item, batch of 32 pages) pairs are walked as one sequence: `cur` holds the batch being
    // consumed, `nxt` the one after it, which may already belong to the next item.
    int2 nxt = first_pages;
    for (int idx = item_begin; idx < item_end && ok; ++idx) {
      const DeviceItem it = get_item(c, misc, idx, item_begin);
      const int n_tiles = (it.n_pages + 7) >> 3;
      int2 cur = make_int2(0, 0);
      for (int t = 0; t < n_tiles && ok; ++t, ++g) {
        if ((t & 3) == 0) {
          cur = nxt;
          nxt = make_int2(0, 0);
          const int ahead = (t + 4) * 8 + lane;
          if ((t + 4) * 8 < it.n_pages) {
            if (ahead < it.n_pages) nxt = c.pd.visit[it.page0 + ahead];
          } else if (idx + 1 < item_end) {          // first batch of the next item
            const DeviceItem nx = get_item(c, misc, idx + 1, item_begin);
            if (lane < nx.n_pages) nxt = c.pd.visit[nx.page0 + lane];
          }
        }
        const int npg = min(8, it.n_pages - t * 8), sl = g & 1;
        int2 pg;
        pg.x = __shfl_sync(0xffffffffu, cur.x, (t & 3) * 8 + (lane & 7));
        pg.y = __shfl_sync(0xffffffffu, cur.y, (t & 3) * 8 + (lane & 7));
        if (lane >= npg) pg = make_int2(0, 0);
        if (lane < npg && !bounds_ok(c.pd, pg.x, 0, 16)) pg.x = 0;       // checking builds: flagged, page 0 read instead
        if (producer_runs_ahead && !waited && __any_sync(0xffffffffu, ((pg.y >> 8) & 31) != 0)) {
          pdl_wait();                                  // new rows come from the previous kernel (or from this one)
          waited = true;
        }
        if (c.k_new != nullptr && !appended && __any_sync(0xffffffffu, ((pg.y >> 8) & 31) != 0)) {
          // fused append: this tile holds rows that are new this step; the append warp has written
          // (or is writing) them -- wait for it once, before the first such page is copied
          int okw = 1;
          if (lane == 0) okw = mbar_wait(bars + 8 * A_DONE, 0, ab) ? 1 : 0;
          if (!__shfl_sync(0xffffffffu, okw, 0)) { ok = false; break; }
          appended = true;
        }
        const uint32_t full = bars + 8 * ((kv ? V_FULL : K_FULL) + sl), empty = bars + 8 * ((kv ? V_EMPTY : K_EMPTY) + sl);
        int good = 1;
        if (lane == 0) good = mbar_wait(empty, ((g >> 1) & 1) ^ 1, ab) ? 1 : 0;
        good = __shfl_sync(0xffffffffu, good, 0);
        if (!good) { ok = false; break; }
        if (lane == 0) ASPD_STAMP(c, g, 6 + kv);
        if (c.stagger_start && g <= 1 && (kv | g) != 0) {
          // A CTA with only a few tiles: its four first tiles requested at once (as all 148 CTAs do)
          // would all land together, late.  So the first K tile goes out alone; the first V tile and the
          // second K tile follow when it has landed, the second V tile when the first has.  Only a
          // hint about the order: the wait is short and gives up silently.
          const uint32_t first = bars + 8 * ((kv == 1 && g == 1) ? V_FULL : K_FULL);
          if (lane == 0) {
            const long long t0 = clock64();
            while (!mbar_try(first, 0) && clock64() - t0 < 8000) { }
          }
          __syncwarp();
        }
        if (kv == 0 && lane < 8) misc->nval[g & 3][lane] = pg.y;   // read by the softmax warps of tile g
        __syncwarp();
        if (lane == 0) mbar_expect_tx(full, (uint32_t)npg * 4096u);
        __syncwarp();
        if (lane < npg)
          bulk_copy(base + (kv ? OFF_V : OFF_K) + sl * kTileBytes + lane * 4096,
                    pool + ((size_t)pg.x * c.n_kv_heads + it.kv_head) * 4096, 4096, full);
        if (lane == 0) ASPD_STAMP(c, g, 13 + kv);
      }
    }
  } else if (warp == W_MMA) {
    // =================================== MMA issuer ===================================
    // The tiles of all items form one pipeline: S of tile g is issued before P.V of tile g - 1,
    // also across an item boundary, so the tensor pipe and the softmax warps never drain
    // between items.  The whole warp walks the loops with warp-uniform values (what comes from
    // shared memory is broadcast from lane 0), lane 0 issues the MMAs and commits.
    {
      const uint32_t full_mask = 0xffffffffu;
      const uint32_t tmem_u = __shfl_sync(full_mask, tmem, 0);
      const uint32_t base_u = __shfl_sync(full_mask, base, 0), bars_u = base_u + off_misc;
      struct TileRef { int npg, first, last, qb, ob, item_no; };   // qb: query tile (always 0 in the wide kernel)
      auto q_fill = [](int item_no) { return WIDE ? item_no : item_no >> 1; };   // how often the item's query tile was filled before
      auto wait_all = [&](uint32_t bar, uint32_t parity) { return __all_sync(full_mask, mbar_wait(bar, parity, ab)) != 0; };
      const uint32_t mma_m = c.m64 ? 64u : 128u;
      const uint32_t idesc_pv = instr_desc(128, 1, (c.m64 || c.pv64) ? 64u : 128u);
      auto issue_s = [&](const TileRef& tr, int g) -> bool {
        const int sb = g & 1;
        if (tr.first && !wait_all(bars_u + 8 * (Q_FULL + tr.qb), q_fill(tr.item_no) & 1)) return false;
        if (!wait_all(bars_u + 8 * (K_FULL + sb), (g >> 1) & 1)) return false;
        if (lane == 0) ASPD_STAMP(c, g, 15);
        if (!wait_all(bars_u + 8 * (S_EMPTY + sb), ((g >> 1) & 1) ^ 1)) return false;
        tc_fence_after();
        if (lane == 0) ASPD_STAMP(c, g, 8);
        const uint32_t qbuf = base_u + OFF_Q + tr.qb * kTileBytes, kbuf = base_u + OFF_K + sb * kTileBytes;
        const uint32_t idesc_s = instr_desc((uint32_t)tr.npg * 16u, 0, mma_m);
        // k-step ks covers head_dim elements [16 ks, 16 ks + 16): span ks / 4, 32 bytes per step
        tc_mma_ss_k128_lane0<kHalf, 1024>(tmem_u + COL_S + sb * 128, smem_desc(qbuf, 16, 1024), smem_desc(kbuf, 16, 2048), idesc_s);
        if (lane == 0) ASPD_STAMP(c, g, 9);
        tc_commit_lane0(bars_u + 8 * (S_FULL + sb));
        tc_commit_lane0(bars_u + 8 * (K_EMPTY + sb));
        if (tr.last) tc_commit_lane0(bars_u + 8 * (Q_EMPTY + tr.qb));
        return true;
      };
      auto issue_pv = [&](const TileRef& tr, int g) -> bool {
        if (lane == 0) ASPD_STAMP(c, g, 10);
        if (!wait_all(bars_u + 8 * P_FULL, g & 1)) return false;
        if (lane == 0) ASPD_STAMP(c, g, 11);
        if (!wait_all(bars_u + 8 * (V_FULL + (g & 1)), (g >> 1) & 1)) return false;
        if (tr.first && !wait_all(bars_u + 8 * (O_EMPTY + tr.ob), ((tr.item_no >> 1) & 1) ^ 1)) return false;
        tc_fence_after();
        const uint32_t pbuf = base_u + OFF_P, vbuf = base_u + OFF_V + (g & 1) * kTileBytes;
        // 16 keys = one page per k-step
        tc_mma_ss_pv_lane0<kHalf>(tmem_u + COL_O + tr.ob * 128, smem_desc(pbuf, 16, 1024), smem_desc(vbuf, 1024, 2048), idesc_pv,
                                  tr.first ? 0u : 1u, tr.npg);
        if (lane == 0) ASPD_STAMP(c, g, 12);
        tc_commit_lane0(bars_u + 8 * P_EMPTY);
        tc_commit_lane0(bars_u + 8 * (V_EMPTY + (g & 1)));
        if (tr.last) tc_commit_lane0(bars_u + 8 * (O_FULL + tr.ob));
        return true;
      };
      int g = 0, item_no = 0;
      bool ok = true, have_prev = false;
      TileRef prev = {0, 0, 0, 0, 0, 0};
      const int ib = __shfl_sync(full_mask, item_begin, 0), ie = __shfl_sync(full_mask, item_end, 0);
      for (int idx = ib; idx < ie && ok; ++idx, ++item_no) {
        const int n_pages = __shfl_sync(full_mask, get_item(c, misc, idx, ib).n_pages, 0), n_tiles = (n_pages + 7) >> 3;
        for (int t = 0; t < n_tiles && ok; ++t, ++g) {
          const TileRef cur = {min(8, n_pages - t * 8), t == 0, t == n_tiles - 1, WIDE ? 0 : item_no & 1, item_no & 1, item_no};
          ok = issue_s(cur, g);
          if (ok && have_prev) ok = issue_pv(prev, g - 1);
          prev = cur;
          have_prev = true;
        }
      }
      if (ok && have_prev) issue_pv(prev, g - 1);
    }
    __syncwarp();
  } else if (warp >= W_EPI) {
    // ===================================== epilogue =====================================
    // One (m, l, O) record per query row of every item, written while the other warps are
    // already working on the next item (O and the statistics are double-buffered by item).
    const int et = tid - W_EPI * 32, ew = warp - W_EPI;   // TMEM lane quadrant = warp % 4 = ew
    const int G = c.n_q_heads / c.n_kv_heads;
    int item_no = 0;
    bool dead = false;
    if (c.k_new != nullptr) append_new_rows(c, et, dirty0, dirty_units, dirty_first);
    mbar_arrive(bars + 8 * A_DONE);
    if (item_begin < item_end) {                   // the first query tile, while the first K/V tiles are in flight
      prep_q(c, get_item(c, misc, item_begin, item_begin), base + OFF_Q, et);
      if constexpr (WIDE) prep_q(c, get_item(c, misc, item_begin, item_begin), base + OFF_Q, et, 512);
      fence_async_smem();
      mbar_arrive(bars + 8 * Q_FULL);
    }
    for (int idx = item_begin; idx < item_end; ++idx, ++item_no) {
      const DeviceItem it = get_item(c, misc, idx, item_begin);
      const bool m64 = !WIDE && (c.m64 || c.pv64);  // O from an M = 64 MMA: row 16 q + i sits in lane i < 16 of quadrant q
      const int ob = item_no & 1, M = it.n_q_tok * G, R = M <= 32 ? 32 : (M <= 64 ? 64 : 128),
                KS = ((!WIDE && c.m64) ? 64 : 128) / R;                // replicas in the softmax threads' layout
      if (idx + 1 < item_end) {                    // the next item's query tile: into the other buffer, or (wide
        const int qn = WIDE ? 0 : (item_no + 1) & 1;   // kernel) into the only one once this item's last S is issued
        const int fills = WIDE ? item_no + 1 : (item_no + 1) >> 1;
        if constexpr (WIDE) {
          // the only query tile is free once this item's last S has been issued: rotate the next
          // item's rows into registers first, so that only the stores are left for after the wait
          const DeviceItem nx = get_item(c, misc, idx + 1, item_begin);
          QUnits q0, q1;
          prep_q_compute(c, nx, et, 0, q0);
          prep_q_compute(c, nx, et, 512, q1);
          dead |= !mbar_wait(bars + 8 * (Q_EMPTY + qn), (fills & 1) ^ 1, ab);
          prep_q_store(c, nx, base + OFF_Q, et, 0, q0);
          prep_q_store(c, nx, base + OFF_Q, et, 512, q1);
        } else {
          dead |= !mbar_wait(bars + 8 * (Q_EMPTY + qn), (fills & 1) ^ 1, ab);
          prep_q(c, get_item(c, misc, idx + 1, item_begin), base + OFF_Q + qn * kTileBytes, et);
        }
        fence_async_smem();
        mbar_arrive(bars + 8 * (Q_FULL + qn));
      }
      dead |= !mbar_wait(bars + 8 * (E_FULL + ob), (item_no >> 1) & 1, ab);
      dead |= !mbar_wait(bars + 8 * (O_FULL + ob), (item_no >> 1) & 1, ab);
      tc_fence_after();
      // where the item's result goes: a record for the merge, or -- when the item is the row's whole key
      // stream -- the normalised output itself
      // (the wide variant only serves plans that deal whole streams: always direct, never a merge)
      const bool merging = !WIDE && c.merge_out != nullptr;
      const bool direct = c.out != nullptr || (merging && it.n_parts == 1);
      __nv_bfloat16* const out_base = c.out != nullptr ? c.out : c.merge_out;
      if (ew < R / (m64 ? 16 : 32)) {
        const int r = m64 ? ((et & 31) < 16 ? ew * 16 + (et & 31) : 1 << 20) : et;   // row of O held by this thread's TMEM lane
        size_t rec = 0;
        if (r < M && !direct) {
          const int tok = it.q_tok0 + r / G;
          rec = (size_t)(c.pd.part_base[tok * c.n_kv_heads + it.kv_head] + it.part_slot) * G + r % G;
          float lt = 0.f;
          for (int jj = 0; jj < KS; ++jj) lt += misc->fin_l[ob][jj * R + r] + misc->fin_l[ob][128 + jj * R + r];
          float mr = R == 128 ? reinterpret_cast<const float*>(misc + 1)[ob * 128 + r] : misc->fin_m[ob][r];
          if (lt == 0.f) mr = -INFINITY;           // no visible key in this item (the wide variant's reference starts at 0)
          if (!dead) c.pd.ws_ml[rec] = make_float2(mr, lt);
        }
        const uint32_t o_addr = tmem + ((uint32_t)(ew * 32) << 16) + COL_O + ob * 128;
        float inv_l = 0.f;                         // direct output: the item is the row's whole key stream
        __nv_bfloat16* orow = nullptr;
        if (direct && r < M) {
          float lt = 0.f;
          for (int jj = 0; jj < KS; ++jj) lt += misc->fin_l[ob][jj * R + r] + misc->fin_l[ob][128 + jj * R + r];
          inv_l = lt > 0.f ? 1.f / lt : 0.f;
          orow = out_base + ((size_t)(it.q_tok0 + r / G) * c.n_q_heads + it.kv_head * G + r % G) * 128;
        }
#pragma unroll 1
        for (int q4 = 0; q4 < 4; ++q4) {
          float o[32];
          ASPD_TMEM_LD32(o_addr + q4 * 32, o, 0);
          tmem_wait_ld();
          if (direct) {
            if (r < M && !dead) {
              uint4* dst = reinterpret_cast<uint4*>(orow + q4 * 32);
#pragma unroll
              for (int i = 0; i < 4; ++i)
                dst[i] = make_uint4(pack_bf16(o[8 * i] * inv_l, o[8 * i + 1] * inv_l), pack_bf16(o[8 * i + 2] * inv_l, o[8 * i + 3] * inv_l),
                                    pack_bf16(o[8 * i + 4] * inv_l, o[8 * i + 5] * inv_l), pack_bf16(o[8 * i + 6] * inv_l, o[8 * i + 7] * inv_l));
            }
          } else if (r < M && !dead) {
            float4* dst = reinterpret_cast<float4*>(c.pd.ws_o + rec * 128 + q4 * 32);
#pragma unroll
            for (int i = 0; i < 8; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bars + 8 * (O_EMPTY + ob));
      if (merging && !direct) {
        // Announce the item's records: every thread's stores are fenced, then one thread per token
        // counts the record in; the thread that counts the last record of a (token, KV head) queues
        // the pair for the merge and puts the counter back to zero for the next launch.  Nobody waits.
        if (et == 0) ASPD_CTA_STAMP(c, 4);
        __threadfence();
        if (misc->mq_n + it.n_q_tok > kMergeQueue) {              // no room for this item's pairs: merge what is queued now
          drain_merge_queue(c, misc, ew, 4, lane);
          named_sync(2, 128);
          if (et == 0) misc->mq_n = 0;
        }
        named_sync(2, 128);
        if (et == 0) ASPD_CTA_STAMP(c, 5);
        if (et < it.n_q_tok && !dead) {
          const int idx = (it.q_tok0 + et) * c.n_kv_heads + it.kv_head;
          if (atomicAdd(c.pd.arrive + idx, 1) == it.n_parts - 1) {
            __threadfence();                                        // the other CTAs' records, before anyone here reads them
            c.pd.arrive[idx] = 0;
            const int e = atomicAdd(&misc->mq_n, 1);
            misc->mq[e][0] = idx; misc->mq[e][1] = c.pd.part_base[idx]; misc->mq[e][2] = it.n_parts;
          }
        }
        if (et == 0) ASPD_CTA_STAMP(c, 6);
      }
      if (named_sync_or(2, 128, dead || *ab)) break;
    }
    if (et == 0) ASPD_CTA_STAMP(c, 2);
  }

  // ---- drain: on a time-out give outstanding copies and MMAs time to land before the CTA's
  // shared memory and TMEM go away
  if (*ab) {
    if (tid == 0) atomicCAS(c.pd.status, 0, (int)ASPD_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0) ASPD_CTA_STAMP(c, 3);
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
  // single-launch plans: the pairs whose last record this CTA stored are merged now, by all warps
  if (!WIDE && c.merge_out != nullptr && !*ab) drain_merge_queue(c, misc, warp, kThreads / 32, lane);
  if (tid == 0) ASPD_CTA_STAMP(c, 7);
}


// A wait that nothing ever satisfies, with a caller-given limit: exercises the bounded-wait path
// (give up, record the status, leave the context usable) without hanging anything.
__global__ void wait_probe_kernel(long long limit_cycles, int32_t* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, limit_cycles);   // nobody arrives
    *status = ok ? (int)ASPD_OK : (int)ASPD_ERR_TIMEOUT;
  }
}

}  // namespace

#include "aspd_attn_tc_w2.cuh"

int launch_wait_probe(long long limit_cycles, int32_t* status_dev, cudaStream_t s) {
  wait_probe_kernel<<<1, 32, 0, s>>>(limit_cycles, status_dev);
  return cudaGetLastError() == cudaSuccess ? ASPD_OK : ASPD_ERR_CUDA;
}

// where the profiling build's stamps go (aspd_debug_profile)
#ifdef ASPD_TC_PROFILE
static long long* g_prof_buf = nullptr;
static int g_prof_cta = 0;
#endif

int set_profile_buffer(long long* device_buf, int cta) {
#ifdef ASPD_TC_PROFILE
  g_prof_buf = device_buf;
  g_prof_cta = cta;
  return ASPD_OK;
#else
  (void)device_buf; (void)cta;
  return ASPD_ERR_UNSUPPORTED;
#endif
}

static int launch_tc(const aspd_plan* p, const void* q, const void* k_new, const void* v_new, const void* k_pool,
                     const void* v_pool, void* out, cudaStream_t s) {
  if (p->n_items == 0) return ASPD_OK;
  const aspd_shape_t& sh = p->shape;
  // the attribute belongs to the (function, device) pair: set it once on every device that launches
  static bool configured[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ASPD_ERR_CUDA;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    if (cudaFuncSetAttribute(attn_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(attn_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(attn_tc_w2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytesW2) != cudaSuccess)
      return ASPD_ERR_CUDA;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  Ctx c;
  c.pd = p->dev;
  c.prof = nullptr;
  c.prof_cta = 0;
#ifdef ASPD_TC_PROFILE
  c.prof = g_prof_buf;
  c.prof_cta = g_prof_cta;
#endif
  c.q = (const __nv_bfloat16*)q;
  c.k_new = (const __nv_bfloat16*)k_new;
  c.v_new = (const __nv_bfloat16*)v_new;
  c.k_pool = (const char*)k_pool;
  c.v_pool = (const char*)v_pool;
  c.n_items = p->n_items;
  c.n_q_heads = sh.n_q_heads;
  c.n_kv_heads = sh.n_kv_heads;
  c.scale_log2 = sh.sm_scale * kLog2e;
  c.early_fetch = p->stable_cache;
  c.stagger_start = p->stagger_start;
  c.m64 = (p->m64 == 1 && !p->wide && !p->dealt) ? 1 : 0;
  c.pv64 = (p->m64 == 2 && !p->wide && !p->dealt) ? 1 : 0;
  c.out = p->dealt ? (__nv_bfloat16*)out : nullptr;   // only when every (token, KV head) has a single item
  c.merge_out = (!p->dealt && p->single_launch) ? (__nv_bfloat16*)out : nullptr;
  if (p->wide == 2) {                       // row blocks of two query tiles: final outputs only
    if (c.out == nullptr) return ASPD_ERR_UNSUPPORTED;
    c.k_new = nullptr; c.v_new = nullptr;
    return launch_pdl(kPdlAttn, attn_tc_w2_kernel, dim3(p->n_ctas), dim3(kThreads), kSmemBytesW2, s, c) == cudaSuccess ? ASPD_OK : ASPD_ERR_CUDA;
  }
  const cudaError_t e = p->wide ? launch_pdl(kPdlAttn, attn_tc_kernel<true>, dim3(p->n_ctas), dim3(kThreads), kSmemBytes, s, c)
                                : launch_pdl(kPdlAttn, attn_tc_kernel<false>, dim3(p->n_ctas), dim3(kThreads), kSmemBytes, s, c);
  return e == cudaSuccess ? ASPD_OK : ASPD_ERR_CUDA;
}

int launch_attn_mma(const aspd_plan* p, const void* q, const void* k_pool, const void* v_pool, void* out, cudaStream_t s) {
  return launch_tc(p, q, nullptr, nullptr, k_pool, v_pool, out, s);
}

int launch_attn_mma_step(const aspd_plan* p, const void* q, const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                         void* out, cudaStream_t s) {
  return launch_tc(p, q, k_new, v_new, k_pool, v_pool, out, s);
}

}  // namespace aspd
