// The two-tile variant of the tensor-core attention kernel (plans that deal whole streams with row
// blocks of up to 256 query rows: masked prefill, teacher forcing).  Included by aspd_attn_tc.cu.
//
// A row block is two query tiles of 128 rows (tile j holds tokens j * (128 / G) ...).  Every K/V
// tile the CTA fetches is scored against both:
//
//     S_j = Q_j . K^T        tcgen05.mma M=128, N=keys, K=128       TMEM columns 128 j
//     softmax group j        four warps, thread r = row r of tile j: the tile's keys in two halves of
//                            64, exponentials against the row's reference maximum (raised only when
//                            an exponent passes 2^40, decided by the thread alone: no exchange), P half
//                            (64 keys, bf16) over the first 32 columns of the half's own scores
//     O_j += P_j . V         tcgen05.mma M=128, N=128, K=64 per half, A operand from tensor memory
//                            TMEM columns 256 + 128 j
//
// so that while one group is in its exponentials the tensor pipe works for the other, and a thread
// owns its row from the first score to the normalised output (it divides by l and stores the row
// itself; there are no statistics to hand over).  Each of the four streams of MMAs (scores and P.V of
// either group) has a warp of its own that takes its operations in order and waits for each one's
// operands.  Warp roles: 0-3 group 0, 4-7 group 1, 8 / 11 K / V producers, 9 / 10 P.V issuers of group
// 0 / 1, 12-15 query preparation, of which 12 / 13 also issue the scores of group 0 / 1 (an item's
// query tiles are written and its scores issued at different times).  Single buffers for S (by halves)
// and the query tiles; K and V tiles double-buffered.  All waits are bounded as in the other variants.
#pragma once

namespace {      // included inside namespace aspd

constexpr uint32_t W2_OFF_K = 0, W2_OFF_V = 2 * kTileBytes, W2_OFF_Q = 4 * kTileBytes, W2_OFF_P = 6 * kTileBytes,
                   W2_OFF_MISC = 7 * kTileBytes;
constexpr uint32_t kPHalfBytes = 16384;       // 128 rows x 64 keys x 2 B: one 128-byte-swizzle span
constexpr size_t kSmemBytesW2 = 7 * kTileBytes + 2048 + 1024;   // + Misc + slack to align the base to 1024
constexpr int kItemCacheW2 = 8;
constexpr bool kPolyExp = true;     // plain pass: a quarter of the exponentials as a cubic on the FMA pipe (10 % fewer cycles per tile;
                                    // under the power cap, same box: none 894-899 us, an eighth 881-882, a quarter 873-879, half 923-928)
constexpr bool kPInTmem = true;    // P halves go into the first 32 columns of their own score half in tensor memory and are the
                                   // A operand of P.V from there (no shared-memory round trip); needs kSplitS
constexpr bool kSplitS = true;     // scores of a tile as two MMAs of 64 keys (own columns and barriers each: a half's columns are
                                   // free again as soon as its pass is final) or one of 128 (measured: 1141 against 1021 us)
// The reference maximum of a row is raised when an exponent passes 2^40 (everything is floating point,
// bf16 and fp32 alike, so the distance costs no precision; what must not happen is an overflow, and
// 2^40 x 2^13 keys x |v| is far from one).  The one-tile variants raise at 2^8.
constexpr float kRaiseW2 = 40.0f, kRaiseSumW2 = 1099511627776.0f;

// S_FULL / S_EMPTY / P_FULL: one per (group, half of the tile's keys)
enum BarW2 { WK_FULL = 0, WK_EMPTY = 2, WV_FULL = 4, WV_EMPTY = 6, WS_FULL = 8, WS_EMPTY = 12, WP_FULL = 16, WP_EMPTY = 20,
             WO_FULL = 22, WQ_FULL = 24, WQ_EMPTY = 25, W2_NUM_BARS = 26 };

static_assert(kSplitS || !kPInTmem, "P in tensor memory lives in its own score half: the scores must be issued by halves");

struct MiscW2 {
  uint64_t bars[W2_NUM_BARS];
  int nval[4][8];                    // page entries of the 8 pages of a tile (ring over 4 tiles)
  DeviceItem items[kItemCacheW2];
  uint32_t tmem_base;
  int abort_flag;
  int lead[2];                       // [1]: the item group 0's P.V issuer is at (read by group 1's); [0] unused
};
static_assert(sizeof(MiscW2) <= 2048, "MiscW2 must fit behind the tiles");

__device__ __forceinline__ DeviceItem get_item_w2(const Ctx& c, const MiscW2* misc, int idx, int item_begin) {
  const int rel = idx - item_begin;
  return rel < kItemCacheW2 ? misc->items[rel] : c.pd.items[idx];
}

// One softmax group over all items of the CTA.  grp = 0 / 1, r = the thread's row in its tile.
__device__ __forceinline__ void softmax_group_w2(const Ctx& c, MiscW2* misc, uint32_t bars, uint32_t base, uint32_t tmem, int item_begin,
                                                 int item_end, int grp, int tpt) {
  const int tid = threadIdx.x, warp = tid >> 5, r = tid & 127;
  const int G = c.n_q_heads / c.n_kv_heads;
  volatile int* ab = &misc->abort_flag;
  const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
  const uint32_t s_base = tmem + lane_addr + COL_S + grp * 128, o_base = tmem + lane_addr + COL_O + grp * 128;
  const uint32_t pbuf = base + W2_OFF_P + grp * kPHalfBytes;
  const uint32_t bar_sfull = bars + 8 * (WS_FULL + 2 * grp), bar_sempty = bars + 8 * (WS_EMPTY + 2 * grp),   // + 8 h
                 bar_pfull = bars + 8 * (WP_FULL + 2 * grp), bar_pempty = bars + 8 * (WP_EMPTY + grp), bar_ofull = bars + 8 * (WO_FULL + grp);
  int g = 0;            // tiles of the CTA so far (both groups count the same)
  int sc[2] = {0, 0}, hc = 0, ic = 0;   // this group's score halves (first / second), P halves and items so far
  bool dead = false;
  for (int idx = item_begin; idx < item_end; ++idx) {
    const DeviceItem it = get_item_w2(c, misc, idx, item_begin);
    const int n_tiles = (it.n_pages + 7) >> 3;
    const int n_tok = min(tpt, it.n_q_tok - grp * tpt);
    if (n_tok <= 0) { g += n_tiles; continue; }                // the block has no second tile
    const int M = n_tok * G, tok = it.q_tok0 + grp * tpt + r / G;
    int4 vis = make_int4(0, 0, 0, 0);                          // padding rows see nothing
    if (r < M) vis = c.pd.tok_vis[tok];
    float m_ref = 0.f, l = 0.f;                                 // see the one-tile variant: the reference starts at 0
    bool seen = r >= M;                                         // padding rows never need the tracking pass
    bool warp_seen = false;                                     // all rows of the warp have (kept up in the full path only)
    for (int t = 0; t < n_tiles; ++t, ++g) {
      const int npg = min(8, it.n_pages - t * 8), halves = npg > 4 ? 2 : 1;
      // the tile's page entries, taken when its first scores are there: the ring slot may be rewritten
      // while this group is still in its pass (the other group, alone in later items, can run several
      // tiles ahead)
      if (!mbar_test(bar_sfull, sc[0] & 1)) dead |= !mbar_wait(bar_sfull, sc[0] & 1, ab);
      int ye8[8];
      {
        const int4 ya = *reinterpret_cast<const int4*>(&misc->nval[g & 3][0]), yb = *reinterpret_cast<const int4*>(&misc->nval[g & 3][4]);
        ye8[0] = ya.x; ye8[1] = ya.y; ye8[2] = ya.z; ye8[3] = ya.w; ye8[4] = yb.x; ye8[5] = yb.y; ye8[6] = yb.z; ye8[7] = yb.w;
      }
      // Most halves lie wholly inside what every row of the warp may see (the prefix, full pages): the
      // warp then takes the pass without any mask arithmetic.  Both halves' verdicts are taken here.
      const int kbt = it.key0 + t * kTile;
      const bool plain0 = r >= M || (kbt + 64 <= vis.x && (ye8[0] & 255) + (ye8[1] & 255) + (ye8[2] & 255) + (ye8[3] & 255) == 64);
      const bool plain1 = r >= M || (kbt + 128 <= vis.x && (ye8[4] & 255) + (ye8[5] & 255) + (ye8[6] & 255) + (ye8[7] & 255) == 64);
      const bool masked0 = __any_sync(0xffffffffu, !plain0), masked1 = __any_sync(0xffffffffu, !plain1);
      for (int h = 0; h < halves; ++h, ++hc) {
        // The scores of the two halves are separate MMAs into separate columns: a half's columns are
        // given back as soon as its pass is final, so its next scores are there before they are needed.
        if (kSplitS && h > 0 && !mbar_test(bar_sfull + 8 * h, sc[h] & 1)) dead |= !mbar_wait(bar_sfull + 8 * h, sc[h] & 1, ab);    // h = 0: waited for above
        if (kSplitS || h == 0) {
          ++sc[h];
          tc_fence_after();
        }
        if (tid == 0) ASPD_STAMP(c, g, 4 * h);
        uint32_t pk[32];
        float tile_sum, tmax;
        // p = 2^(s * scale - ref) for the thread's 64 scores of this half.  The common pass does not
        // track the largest exponent: packed fp32 pairs (one FFMA and one FADD per two scores), the
        // exponentials, the bf16 pairs.  An exponent beyond 2^40 shows in the sum; the tracking pass
        // then (and for rows that have not seen a key yet) finds the maximum.
        const int kb0 = kbt + h * 64;
        const bool masked = h ? masked1 : masked0;
        auto pass_impl = [&](float ref, auto track_tag, auto masked_tag) {
          constexpr bool TRACK = decltype(track_tag)::value, MASKED = decltype(masked_tag)::value;
          float mx0 = -INFINITY, mx1 = -INFINITY;
          float2 sum0 = make_float2(0.f, 0.f), sum1 = sum0, sum2 = sum0, sum3 = sum0;
          const float2 sc2 = make_float2(c.scale_log2, c.scale_log2), nb2 = make_float2(-ref, -ref);
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {
            float s[32];
            ASPD_TMEM_LD32(s_base + h * 64 + ch * 32, s, 0);
            tmem_wait_ld();
#pragma unroll
            for (int pg = 0; pg < 2; ++pg) {
              const int nv = (h ? ye8[4 + ch * 2 + pg] : ye8[ch * 2 + pg]) & 255;
              const int kb = it.key0 + t * kTile + h * 64 + ch * 32 + pg * 16;
              uint32_t mask = 0xFFFFu;
              if constexpr (MASKED) mask = bits_between(0, min(nv, vis.x - kb)) | bits_between(vis.y - kb, min(nv, vis.z - kb));
#pragma unroll
              for (int i = 0; i < 16; i += 4) {
                float2 x0 = __ffma2_rn(make_float2(s[pg * 16 + i], s[pg * 16 + i + 1]), sc2, nb2);
                float2 x1 = __ffma2_rn(make_float2(s[pg * 16 + i + 2], s[pg * 16 + i + 3]), sc2, nb2);
                if (MASKED && mask != 0xFFFFu) {
                  x0.x = (mask >> i) & 1u ? x0.x : -INFINITY;
                  x0.y = (mask >> (i + 1)) & 1u ? x0.y : -INFINITY;
                  x1.x = (mask >> (i + 2)) & 1u ? x1.x : -INFINITY;
                  x1.y = (mask >> (i + 3)) & 1u ? x1.y : -INFINITY;
                }
                if constexpr (TRACK) { mx0 = fmaxf(mx0, fmaxf(x0.x, x0.y)); mx1 = fmaxf(mx1, fmaxf(x1.x, x1.y)); }
                // in the plain pass a quarter of the exponentials goes to the FMA pipe
                x0.x = ex2(x0.x); x0.y = ex2(x0.y);
                if (kPolyExp && !TRACK && !MASKED && (i & 4)) x1 = ex2_fma2(x1);
                else { x1.x = ex2(x1.x); x1.y = ex2(x1.y); }
                if (i & 4) { sum2 = __fadd2_rn(sum2, x0); sum3 = __fadd2_rn(sum3, x1); }
                else       { sum0 = __fadd2_rn(sum0, x0); sum1 = __fadd2_rn(sum1, x1); }
                pk[ch * 16 + pg * 8 + (i >> 1)] = pack_bf16(x0.x, x0.y);
                pk[ch * 16 + pg * 8 + (i >> 1) + 1] = pack_bf16(x1.x, x1.y);
              }
            }
          }
          const float2 st = __fadd2_rn(__fadd2_rn(sum0, sum1), __fadd2_rn(sum2, sum3));
          tile_sum = st.x + st.y;
          tmax = fmaxf(mx0, mx1);
        };
        auto pass = [&](float ref, auto track_tag) {
          if (masked) pass_impl(ref, track_tag, std::true_type());
          else pass_impl(ref, track_tag, std::false_type());
        };
        // The common case -- every row of the warp has seen a key and no exponent passed 2^40 -- is
        // the plain pass and one vote; everything else goes the full way.
        bool settled = false;
        if (warp_seen) {
          pass(m_ref, std::false_type());
          // an exponent beyond 2^40 makes the sum exceed it (the converse is harmless: one more pass)
          settled = !__any_sync(0xffffffffu, !(tile_sum <= kRaiseSumW2));
        }
        if (!settled) {
          pass(m_ref, std::true_type());
          // move the reference: up when an exponent passed 2^40; down only while the row has not seen a
          // key yet (l and its row of O are still exactly 0 then, so nothing is rescaled)
          const bool raise = tmax > kRaiseW2, lower = !seen && tmax < -kLower && tmax > -INFINITY;
          const bool upd = raise || lower;
          seen |= tmax > -INFINITY;
          warp_seen = !__any_sync(0xffffffffu, !seen);
          float alpha = 1.f;
          if (raise) alpha = ex2(-tmax);
          if (upd) m_ref += tmax;
          l *= alpha;
          if (__any_sync(0xffffffffu, upd)) {
            if (t > 0 || h > 0) {                     // the rows' O so far is rescaled in TMEM (the warp together)
              dead |= !mbar_wait(bar_pempty, (hc - 1) & 1, ab);      // the P.V of the previous half is done
              tc_fence_after();
#pragma unroll 1
              for (int q4 = 0; q4 < 4; ++q4) {
                float o[32];
                ASPD_TMEM_LD32(o_base + q4 * 32, o, 0);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] *= alpha;
                ASPD_TMEM_ST32(o_base + q4 * 32, o, 0);
              }
              tmem_wait_st();
            }
            pass(m_ref, std::false_type());           // the whole warp again (TMEM loads are warp-wide)
          }
        }
        l += tile_sum;
        if (!kPInTmem && (kSplitS || h == halves - 1)) {   // the scores are read: the MMA warp may overwrite them
          tc_fence_before();
          mbar_arrive(bar_sempty + (kSplitS ? 8 * h : 0));
        }
        if (tid == 0) ASPD_STAMP(c, g, 4 * h + 1);
        if constexpr (kPInTmem) {
          // the half's P (64 bf16 = 32 columns) over its own scores, which nobody needs any more: the
          // MMA warp frees these columns for the next tile's scores when this half's P.V is done
          ASPD_TMEM_ST32U(s_base + h * 64, pk, 0);
          tmem_wait_st();
          // (each half has its own barrier: the scores that P replaces were issued only after the
          // half's previous P.V was done, so its previous announcement has been taken)
          if (tid == 0) ASPD_STAMP(c, g, 4 * h + 2);
        } else {
          if (hc > 0) dead |= !mbar_wait(bar_pempty, (hc - 1) & 1, ab);   // the P half buffer is free again
          if (tid == 0) ASPD_STAMP(c, g, 4 * h + 2);
#pragma unroll
          for (int c8 = 0; c8 < 8; ++c8) {
            const uint32_t addr = pbuf + r * 128 + ((c8 ^ (r & 7)) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pk[c8 * 4 + 0]), "r"(pk[c8 * 4 + 1]),
                         "r"(pk[c8 * 4 + 2]), "r"(pk[c8 * 4 + 3]) : "memory");
          }
          fence_async_smem();
        }
        tc_fence_before();
        mbar_arrive(bar_pfull + (kPInTmem ? 8 * h : 0));
        if (tid == 0) ASPD_STAMP(c, g, 4 * h + 3);
      }
    }
    // ---- the row is complete: normalise and store it
    dead |= !mbar_wait(bar_ofull, ic & 1, ab);
    tc_fence_after();
    ++ic;
    {
      const float inv_l = l > 0.f ? 1.f / l : 0.f;
      __nv_bfloat16* orow = c.out + ((size_t)tok * c.n_q_heads + it.kv_head * G + r % G) * 128;
#pragma unroll 1
      for (int q4 = 0; q4 < 4; ++q4) {
        float o[32];
        ASPD_TMEM_LD32(o_base + q4 * 32, o, 0);
        tmem_wait_ld();
        if (r < M && !dead) {
          uint4* dst = reinterpret_cast<uint4*>(orow + q4 * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i)
            dst[i] = make_uint4(pack_bf16(o[8 * i] * inv_l, o[8 * i + 1] * inv_l), pack_bf16(o[8 * i + 2] * inv_l, o[8 * i + 3] * inv_l),
                                pack_bf16(o[8 * i + 4] * inv_l, o[8 * i + 5] * inv_l), pack_bf16(o[8 * i + 6] * inv_l, o[8 * i + 7] * inv_l));
        }
      }
      tc_fence_before();
    }
    if (named_sync_or(1 + grp, 128, dead || *ab)) break;
  }
}


__global__ void __launch_bounds__(kThreads, 1) attn_tc_w2_kernel(Ctx c) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  MiscW2* misc = reinterpret_cast<MiscW2*>(smem + W2_OFF_MISC);
  const uint32_t bars = base + W2_OFF_MISC;       // bars[] is the first member
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* ab = &misc->abort_flag;
  if (tid == 0) ASPD_CTA_STAMP(c, 0);
  if (tid == 0) pdl_launch_dependents();
  const int4 head = c.pd.cta_head[blockIdx.x];
  const int item_begin = head.x, item_end = head.y;
  int2 first_pages = make_int2(0, 0);
  if ((warp == W_KPROD || warp == W_VPROD) && lane < head.w) first_pages = c.pd.visit[head.z + lane];
  {
    const int n_cached = min(item_end - item_begin, kItemCacheW2);
    for (int e = tid; e < n_cached * (int)(sizeof(DeviceItem) / 4); e += kThreads)
      reinterpret_cast<int*>(misc->items)[e] = reinterpret_cast<const int*>(c.pd.items + item_begin)[e];
  }
  if (tid == 0) {
    //                               K_FULL K_EMPTY V_FULL V_EMPTY S_FULL(4)   S_EMPTY(4)          P_FULL(4)           P_EMPTY O_FULL Q_FULL Q_EMPTY
    const int se = kPInTmem ? 1 : 128;      // who gives a score half's columns back: the MMA warp's commit, or the 128 threads that read them
    const int counts[W2_NUM_BARS] = {1, 1,  2, 2,   1, 1,  2, 2,   1, 1, 1, 1,  se, se, se, se, 128, 128, 128, 128, 1, 1,   1, 1,  128,   2};
    for (int i = 0; i < W2_NUM_BARS; ++i) mbar_init(bars + 8 * i, counts[i]);
    misc->abort_flag = 0;
    misc->lead[0] = item_begin; misc->lead[1] = item_begin;
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
  const int G = c.n_q_heads / c.n_kv_heads, tpt = 128 / G;      // tokens per query tile
  // inputs written by earlier kernels of the stream are used from here on; with the plan's
  // stable-cache promise the producers go ahead (such plans never carry new rows in their pages'
  // entries only when the step was appended by an earlier kernel: they wait before the first such page)
  const bool producer_runs_ahead = c.early_fetch && (warp == W_KPROD || warp == W_VPROD);
  if (!producer_runs_ahead) pdl_wait();
  if (tid == 0) ASPD_CTA_STAMP(c, 1);

  if (warp < 8) {
    softmax_group_w2(c, misc, bars, base, tmem, item_begin, item_end, warp >> 2, tpt);
  } else if (warp == W_KPROD || warp == W_VPROD) {
    // ================================ bulk-copy producers (as in the other variants) ================================
    const int kv = warp == W_KPROD ? 0 : 1;
    const char* pool = kv ? c.v_pool : c.k_pool;
    int g = 0;
    bool ok = true, waited = false;
    int2 nxt = first_pages;
    for (int idx = item_begin; idx < item_end && ok; ++idx) {
      const DeviceItem it = get_item_w2(c, misc, idx, item_begin);
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
            const DeviceItem nx = get_item_w2(c, misc, idx + 1, item_begin);
            if (lane < nx.n_pages) nxt = c.pd.visit[nx.page0 + lane];
          }
        }
        const int npg = min(8, it.n_pages - t * 8), sl = g & 1;
        int2 pg;
        pg.x = __shfl_sync(0xffffffffu, cur.x, (t & 3) * 8 + (lane & 7));
        pg.y = __shfl_sync(0xffffffffu, cur.y, (t & 3) * 8 + (lane & 7));
        if (lane >= npg) pg = make_int2(0, 0);
        if (lane < npg && !bounds_ok(c.pd, pg.x, 0, 16)) pg.x = 0;
        if (producer_runs_ahead && !waited && __any_sync(0xffffffffu, ((pg.y >> 8) & 31) != 0)) {
          pdl_wait();                                  // new rows come from the previous kernel
          waited = true;
        }
        const uint32_t full = bars + 8 * ((kv ? WV_FULL : WK_FULL) + sl), empty = bars + 8 * ((kv ? WV_EMPTY : WK_EMPTY) + sl);
        int good = 1;
        if (lane == 0) good = mbar_wait(empty, ((g >> 1) & 1) ^ 1, ab) ? 1 : 0;
        good = __shfl_sync(0xffffffffu, good, 0);
        if (!good) { ok = false; break; }
        if (lane == 0) ASPD_STAMP(c, g, 13 + kv);
        if (kv == 0 && lane < 8) misc->nval[g & 3][lane] = pg.y;   // read by the softmax groups of tile g
        __syncwarp();
        if (lane == 0) mbar_expect_tx(full, (uint32_t)npg * 4096u);
        __syncwarp();
        if (lane < npg)
          bulk_copy(base + (kv ? W2_OFF_V : W2_OFF_K) + sl * kTileBytes + lane * 4096,
                    pool + ((size_t)pg.x * c.n_kv_heads + it.kv_head) * 4096, 4096, full);
      }
    }
  } else if (warp == W_MMA || warp == W_MMA + 1) {
    // ================================ P.V issuers (warp 9: group 0, warp 10: group 1) ================================
    // One warp per stream of operations, each with one cursor and a suspending wait for every
    // operand (all lanes wait, so the warp never diverges; lane 0 issues).  A warp that polled two
    // cursors (scores and P.V of its group) spent ~1300 cycles per operation on asking, issuing and
    // committing, beside two softmax warps on its scheduler, and was what bounded the tile period.
    const int grp = warp - W_MMA;
    const uint32_t fm = 0xffffffffu;
    const uint32_t tmem_u = __shfl_sync(fm, tmem, 0), base_u = __shfl_sync(fm, base, 0), bars_u = base_u + W2_OFF_MISC;
    const int ib = __shfl_sync(fm, item_begin, 0), ie = __shfl_sync(fm, item_end, 0);
    auto wait_all = [&](uint32_t bar, uint32_t parity) { return __all_sync(fm, mbar_wait(bar, parity, ab)) != 0; };
    // A parity only tells the two latest phases of a barrier apart.  Group 1 is absent from items with
    // a single query tile, so its cursor may come to an item that group 0 has not reached yet and
    // would then take an older phase of a V barrier for its own: it holds until group 0's cursor
    // has reached the item (group 0's warp publishes how far it is).
    volatile int* lead = misc->lead;
    const uint32_t idesc_pv = instr_desc(128, 1);
    const uint32_t o_tmem = tmem_u + COL_O + grp * 128, p_tmem = tmem_u + COL_S + grp * 128;
    int gbase = 0, cnt_p[2] = {0, 0};        // P.V operations so far on either half
    bool ok = true;
    for (int idx = ib; idx < ie && ok; ++idx) {
      const DeviceItem it = get_item_w2(c, misc, idx, ib);
      const int n_pages = __shfl_sync(fm, it.n_pages, 0), n_q_tok = __shfl_sync(fm, it.n_q_tok, 0), n_tiles = (n_pages + 7) >> 3;
      if (n_q_tok > grp * tpt) {
        const bool both = n_q_tok > tpt;
        if (grp == 1) {
          const long long t0 = clock64();
          while (ok && __shfl_sync(fm, lead[1], 0) < idx) {
            __nanosleep(100);
            if (__shfl_sync(fm, (*ab || clock64() - t0 > kWaitCycles) ? 1 : 0, 0)) { *ab = 1; ok = false; }
          }
        }
        for (int t = 0; t < n_tiles && ok; ++t) {
          const int g = gbase + t, npg = min(8, n_pages - t * 8), halves = npg > 4 ? 2 : 1;
          const uint32_t vbuf = base_u + W2_OFF_V + (g & 1) * kTileBytes;
          for (int h = 0; h < halves && ok; ++h) {
            const int ph = kPInTmem ? h : 0;
            ok = wait_all(bars_u + 8 * (WP_FULL + 2 * grp + ph), cnt_p[ph] & 1) && (h > 0 || wait_all(bars_u + 8 * (WV_FULL + (g & 1)), (g >> 1) & 1));
            ++cnt_p[ph];
            if (!ok) break;
            tc_fence_after();
            if (lane == 0 && grp == 0 && h == 0) ASPD_STAMP(c, g, 15);
            if constexpr (kPInTmem) {        // 16 keys = one page per k-step
              tc_mma_ts_pv_lane0(o_tmem, p_tmem + h * 64, smem_desc(vbuf + 4 * h * 4096, 1024, 2048), idesc_pv, (t > 0 || h > 0) ? 1u : 0u,
                                 min(4, npg - 4 * h));
            } else {
              const uint32_t pbuf = base_u + W2_OFF_P + grp * kPHalfBytes;
#pragma unroll
              for (int ks = 0; ks < 4; ++ks)
                if (ks < npg - 4 * h)
                  tc_mma_lane0(o_tmem, smem_desc(pbuf + ks * 32, 16, 1024), smem_desc(vbuf + (4 * h + ks) * 4096, 1024, 2048), idesc_pv,
                               (t > 0 || h > 0 || ks > 0) ? 1u : 0u);
            }
            tc_commit_lane0(bars_u + 8 * (WP_EMPTY + grp));
            if constexpr (kPInTmem) tc_commit_lane0(bars_u + 8 * (WS_EMPTY + 2 * grp + h));   // the half's columns are free for the next scores
            if (lane == 0 && grp == 0) ASPD_STAMP(c, g, 10 + h);
            if (h == halves - 1) {
              tc_commit_lane0(bars_u + 8 * (WV_EMPTY + (g & 1)));
              if (!both && lane == 0) mbar_arrive(bars_u + 8 * (WV_EMPTY + (g & 1)));       // the absent group's share
              if (t == n_tiles - 1) tc_commit_lane0(bars_u + 8 * (WO_FULL + grp));
            }
          }
        }
        if (grp == 0 && lane == 0) lead[1] = idx + 1;
      }
      gbase += n_tiles;
    }
    if (grp == 0 && lane == 0) lead[1] = ie;
    __syncwarp();
  } else if (warp >= W_EPI) {
    // ================== query preparation (warps 12-15) and score issuers (warp 12: group 0, warp 13: group 1) ==================
    // The query tiles of an item can be written only when the last scores of the previous item have
    // been issued, and the first scores of an item need its query tiles: the two never overlap, so
    // two of the preparation warps issue the score MMAs between their preparations (one cursor each,
    // suspending waits, the tiles of an item in order).
    const int et = tid - W_EPI * 32, grp = warp - W_EPI;       // grp is a group only for warps 12 and 13
    const uint32_t fm = 0xffffffffu;
    const uint32_t tmem_u = __shfl_sync(fm, tmem, 0), base_u = __shfl_sync(fm, base, 0), bars_u = base_u + W2_OFF_MISC;
    auto wait_all = [&](uint32_t bar, uint32_t parity) { return __all_sync(fm, mbar_wait(bar, parity, ab)) != 0; };
    const uint64_t adesc_q = smem_desc(base_u + W2_OFF_Q + (grp & 1) * kTileBytes, 16, 1024);
    bool dead = false;
    int item_no = 0, gbase = 0, cnt[2] = {0, 0};
    for (int idx = item_begin; idx < item_end; ++idx, ++item_no) {
      const DeviceItem it = get_item_w2(c, misc, idx, item_begin);
      bool waited_q = false;
      for (int j = 0; j < 2; ++j) {
        DeviceItem sub = it;
        sub.q_tok0 = it.q_tok0 + j * tpt;
        sub.n_q_tok = min(tpt, it.n_q_tok - j * tpt);
        if (sub.n_q_tok <= 0) break;
#pragma unroll 1
        for (int e0 = 0; e0 < 1024; e0 += 512) {
          QUnits qu;
          prep_q_compute(c, sub, et, e0, qu, true);
          if (!waited_q) {      // the tiles are free once the previous item's last scores have been issued
            dead |= !mbar_wait(bars + 8 * WQ_EMPTY, (item_no & 1) ^ 1, ab);
            waited_q = true;
          }
          prep_q_store(c, sub, base + W2_OFF_Q + j * kTileBytes, et, e0, qu, true);
        }
      }
      fence_async_smem();
      mbar_arrive(bars + 8 * WQ_FULL);
      if (named_sync_or(3, 128, dead || *ab)) break;
      // ---- S_grp = Q_grp . K^T for the halves of the item's tiles (keys 64 h ... of a tile)
      const int n_pages = __shfl_sync(fm, it.n_pages, 0), n_q_tok = __shfl_sync(fm, it.n_q_tok, 0), n_tiles = (n_pages + 7) >> 3;
      if (grp < 2 && n_q_tok > grp * tpt) {
        const bool both = n_q_tok > tpt;
        bool ok = wait_all(bars_u + 8 * WQ_FULL, item_no & 1);
        for (int t = 0; t < n_tiles && ok; ++t) {
          const int g = gbase + t, sb = g & 1, npg = min(8, n_pages - t * 8), halves = (kSplitS && npg > 4) ? 2 : 1;
          for (int h = 0; h < halves && ok; ++h) {
            ok = (h > 0 || wait_all(bars_u + 8 * (WK_FULL + sb), (g >> 1) & 1)) && wait_all(bars_u + 8 * (WS_EMPTY + 2 * grp + h), (cnt[h] & 1) ^ 1);
            if (!ok) break;
            tc_fence_after();
            const uint32_t kbuf = base_u + W2_OFF_K + sb * kTileBytes + h * 16384;
            const uint32_t idesc_s = instr_desc((uint32_t)(kSplitS ? min(4, npg - 4 * h) : npg) * 16u, 0);
            if (lane == 0 && grp == 0 && h == 0) ASPD_STAMP(c, g, 12);
            tc_mma_ss_k128_lane0<kHalf, 1024>(tmem_u + COL_S + grp * 128 + h * 64, adesc_q, smem_desc(kbuf, 16, 2048), idesc_s);
            tc_commit_lane0(bars_u + 8 * (WS_FULL + 2 * grp + h));
            if (lane == 0 && grp == 0) ASPD_STAMP(c, g, 8 + h);
            ++cnt[h];
            if (h == halves - 1) {
              tc_commit_lane0(bars_u + 8 * (WK_EMPTY + sb));
              if (!both && lane == 0) mbar_arrive(bars_u + 8 * (WK_EMPTY + sb));       // the absent group's share
              if (t == n_tiles - 1) {
                tc_commit_lane0(bars_u + 8 * WQ_EMPTY);
                if (!both && lane == 0) mbar_arrive(bars_u + 8 * WQ_EMPTY);
              }
            }
          }
        }
        dead |= !ok;
      }
      gbase += n_tiles;
    }
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
}

}  // namespace
