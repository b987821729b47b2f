// Probe (development aid, not part of the library): the exponent pass of the two-tile kernel in isolation --
// 64 scores per row from tensor memory, masks, packed scale-and-subtract, ex2, sums, bf16 pairs, P back to
// tensor memory -- by 8 warps (two per SM sub-partition) that do nothing else, with and without the mask
// arithmetic, alone or beside 7 warps in the bounded barrier wait and one that issues MMAs all the time.
// Prints cycles per pass and warp.
#include <cstdio>
#include <cstdlib>
#include <vector>
#include <type_traits>
#include "aspd_tc_common.cuh"
using namespace aspd;
__device__ __forceinline__ uint32_t bits_between(int lo, int hi) {
  lo = max(lo, 0); hi = min(hi, 16);
  return hi > lo ? ((0xFFFFu >> (16 - hi)) & ~((1u << lo) - 1u)) : 0u;
}
template <int MODE, int WAITERS>
__global__ void __launch_bounds__(512, 1) k(int with_mma, const int* nval, const int4* visg, float* out, long long* cyc, int n, float scale) {
  __shared__ uint32_t tmem_base;
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) { abort_flag = 0; mbar_init(smem_u32(&bar), 8); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
  const int tid = threadIdx.x, warp = tid >> 5;
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before(); __syncthreads(); tc_fence_after();
  const uint32_t tmem = tmem_base;
  float l = 0.f;
  if (warp < 8) {
    const int grp = warp >> 2, r = tid & 127;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t s_base = tmem + lane_addr + grp * 128;
    {   // random scores in (-8, 8)
      uint32_t v[32];
      for (int cb = 0; cb < 128; cb += 32) {
        for (int i = 0; i < 32; ++i) { uint32_t x = (tid * 128 + cb + i) * 2654435761u; x ^= x >> 13; x *= 0x5bd1e995u; v[i] = __float_as_uint(((int)(x >> 8) % 4096) * (1.f / 256.f) - 8.f); }
        ASPD_TMEM_ST32U(s_base + cb, v, 0);
      }
      tmem_wait_st();
    }
    const int4 vis = visg[r];
    int ye8[8];
    for (int i = 0; i < 8; ++i) ye8[i] = nval[i];
    const float2 sc2 = make_float2(scale, scale);
    float m_ref = 0.f;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    const long long t0 = clock64();
    for (int it = 0; it < n; ++it) {
      const int h = it & 1, t = it >> 1;
      uint32_t pk[32];
      float tile_sum;
      float2 sum0 = make_float2(0.f, 0.f), sum1 = sum0, sum2 = sum0, sum3 = sum0;
      const float2 nb2 = make_float2(-m_ref, -m_ref);
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        float s[32];
        ASPD_TMEM_LD32(s_base + h * 64 + ch * 32, s, 0);
        tmem_wait_ld();
#pragma unroll
        for (int pg = 0; pg < 2; ++pg) {
          uint32_t mask = 0xFFFFu;
          if (MODE == 0 || MODE == 2) {
            const int nv = (h ? ye8[4 + ch * 2 + pg] : ye8[ch * 2 + pg]) & 255;
            const int kb = t * 128 + h * 64 + ch * 32 + pg * 16;
            mask = bits_between(0, min(nv, vis.x - kb)) | bits_between(vis.y - kb, min(nv, vis.z - kb));
          }
#pragma unroll
          for (int i = 0; i < 16; i += 4) {
            float2 x0, x1;
            if (MODE >= 2) {
              x0.x = fmaf(s[pg * 16 + i], sc2.x, nb2.x); x0.y = fmaf(s[pg * 16 + i + 1], sc2.x, nb2.x);
              x1.x = fmaf(s[pg * 16 + i + 2], sc2.x, nb2.x); x1.y = fmaf(s[pg * 16 + i + 3], sc2.x, nb2.x);
            } else {
              x0 = __ffma2_rn(make_float2(s[pg * 16 + i], s[pg * 16 + i + 1]), sc2, nb2);
              x1 = __ffma2_rn(make_float2(s[pg * 16 + i + 2], s[pg * 16 + i + 3]), sc2, nb2);
            }
            if (MODE == 0 || MODE == 2) {
              if (mask != 0xFFFFu) {
                x0.x = (mask >> i) & 1u ? x0.x : -INFINITY;
                x0.y = (mask >> (i + 1)) & 1u ? x0.y : -INFINITY;
                x1.x = (mask >> (i + 2)) & 1u ? x1.x : -INFINITY;
                x1.y = (mask >> (i + 3)) & 1u ? x1.y : -INFINITY;
              }
            }
            x0.x = ex2(x0.x); x0.y = ex2(x0.y); x1.x = ex2(x1.x); x1.y = ex2(x1.y);
            if (MODE >= 2) { sum0.x += x0.x; sum0.y += x0.y; sum1.x += x1.x; sum1.y += x1.y; }
            else if (i & 4) { sum2 = __fadd2_rn(sum2, x0); sum3 = __fadd2_rn(sum3, x1); }
            else       { sum0 = __fadd2_rn(sum0, x0); sum1 = __fadd2_rn(sum1, x1); }
            pk[ch * 16 + pg * 8 + (i >> 1)] = pack_bf16(x0.x, x0.y);
            pk[ch * 16 + pg * 8 + (i >> 1) + 1] = pack_bf16(x1.x, x1.y);
          }
        }
      }
      const float2 st = __fadd2_rn(__fadd2_rn(sum0, sum1), __fadd2_rn(sum2, sum3));
      tile_sum = st.x + st.y;
      if (__any_sync(0xffffffffu, !(tile_sum <= 1099511627776.0f))) m_ref += 1.f;
      l += tile_sum;
      // P over the second half's columns of the other group's unused area (keeps the scores intact)
      ASPD_TMEM_ST32U(tmem + lane_addr + 256 + grp * 128 + h * 32, pk, 0);
      tmem_wait_st();
    }
    const long long t1 = clock64();
    if ((tid & 31) == 0) { cyc[blockIdx.x * 8 + warp] = t1 - t0; mbar_arrive(smem_u32(&bar)); }
    out[blockIdx.x * 256 + tid] = l;
  }
  if (warp == 9 && with_mma) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const uint32_t abuf = (smem_u32(smem_raw) + 1023u) & ~1023u, bbuf = abuf + 32 * 1024;
    __shared__ __align__(8) unsigned long long mbar2;
    if ((tid & 31) == 0) { mbar_init(smem_u32(&mbar2), 1); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
    __syncwarp();
    uint32_t ph = 0;
    long long nops = 0;
    while (!mbar_test(smem_u32(&bar), 0)) {
      // one tile of both groups: scores into columns 384.. (unused by the passes), P.V from columns 256.. into 448..
      for (int g = 0; g < 2; ++g) {
        tc_mma_ss_k128_lane0<16384, 1024>(tmem + 384, smem_desc(abuf, 16, 1024), smem_desc(bbuf, 16, 2048), instr_desc(64, 0));
        tc_mma_ss_k128_lane0<16384, 1024>(tmem + 384, smem_desc(abuf, 16, 1024), smem_desc(bbuf + 16384, 16, 2048), instr_desc(64, 0));
        tc_mma_ts_pv_lane0(tmem + 384, tmem + 256 + g * 128, smem_desc(bbuf, 1024, 2048), instr_desc(64, 1), 1, 4);
        tc_mma_ts_pv_lane0(tmem + 384, tmem + 256 + g * 128 + 32, smem_desc(bbuf + 16384, 1024, 2048), instr_desc(64, 1), 1, 4);
      }
      tc_commit_lane0(smem_u32(&mbar2));
      __all_sync(0xffffffffu, mbar_wait(smem_u32(&mbar2), ph, &abort_flag));
      ph ^= 1; ++nops;
    }
    if ((tid & 31) == 0) cyc[blockIdx.x * 8 + 7 + 0 * warp] = 0 * nops + cyc[blockIdx.x * 8 + 7];
  }
  if (warp >= 8 && WAITERS && !(warp == 9 && with_mma)) { if (WAITERS == 1) mbar_wait(smem_u32(&bar), 0, &abort_flag); else { bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar), 0, &abort_flag)); if (!ok) abort_flag = 1; } }
  tc_fence_before(); __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}
int main() {
  int* nval; int4* vis; float* out; long long* cyc;
  cudaMalloc(&nval, 32); cudaMalloc(&vis, 128 * 16); cudaMalloc(&out, 148 * 256 * 4); cudaMalloc(&cyc, 148 * 8 * 8);
  int hn[8] = {16, 16, 16, 16, 16, 16, 16, 16}; cudaMemcpy(nval, hn, 32, cudaMemcpyHostToDevice);
  std::vector<int> hv(128 * 4); for (int r = 0; r < 128; ++r) { hv[4 * r] = 1 << 28; hv[4 * r + 1] = 0; hv[4 * r + 2] = 0; hv[4 * r + 3] = 0; }
  cudaMemcpy(vis, hv.data(), 128 * 16, cudaMemcpyHostToDevice);
  const char* names[] = {"masks, alone", "masks, 7 warps waiting and one issuing MMAs all the time", "no masks, alone", "no masks, 7 waiting + MMAs"};
  const int n = 2000;
  cudaFuncSetAttribute(k<0, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024); cudaFuncSetAttribute(k<0, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024); cudaFuncSetAttribute(k<1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024); cudaFuncSetAttribute(k<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
  for (int mode = 0; mode < 4; ++mode) {
    for (int rep = 0; rep < 2; ++rep) {
      if (mode == 0) k<0, 0><<<148, 512, 100 * 1024>>>(0, nval, vis, out, cyc, n, 0.127f);
      if (mode == 1) k<0, 1><<<148, 512, 100 * 1024>>>(1, nval, vis, out, cyc, n, 0.127f);
      if (mode == 2) k<1, 0><<<148, 512, 100 * 1024>>>(0, nval, vis, out, cyc, n, 0.127f);
      if (mode == 3) k<1, 1><<<148, 512, 100 * 1024>>>(1, nval, vis, out, cyc, n, 0.127f);
    }
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { printf("error %s\n", cudaGetErrorString(e)); return 1; }
    long long c[8]; cudaMemcpy(c, cyc, sizeof(c), cudaMemcpyDeviceToHost);
    printf("%-44s: per warp %.0f %.0f %.0f %.0f | %.0f %.0f %.0f %.0f\n", names[mode], (double)c[0] / n, (double)c[1] / n, (double)c[2] / n, (double)c[3] / n, (double)c[4] / n, (double)c[5] / n, (double)c[6] / n, (double)c[7] / n);
  }
  return 0;
}
