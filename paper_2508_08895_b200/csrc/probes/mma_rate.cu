// Probe (development aid, not part of the library): how often tcgen05.mma of the shapes the attention
// kernels use can be issued -- a loop of the same instructions with ready operands, one CTA per SM --
// alone (bg 0), beside four warps of tcgen05.ld (bg 1), beside four warps of shared-memory stores and
// loads (bg 2) or both (bg 3), with zero or random operands.  Prints cycles per MMA.  All waits bounded.
//   usage: mma_rate [CTAs, default 148]
#include <cstdio>
#include <cstdlib>
#include <vector>
#include "aspd_tc_common.cuh"

using namespace aspd;

struct Args {
  int mode;     // 0 S half (N=64), 1 S whole (N=128), 2 N=256, 3 PV SS, 4 PV TS, 5 S whole M=64, 6 mix of a W2 tile: per group 2 x score half + 2 x P.V half with A in tensor memory
  int nrep;     // groups of 8 MMAs
  int bg;       // 0 none, 1 TMEM loads by 8 warps, 2 shared-memory stores+loads by 8 warps, 3 both
  int data;     // 0 zeros, 1 random bf16 in shared and tensor memory
  int chain;    // 1: the 8 MMAs of a group accumulate into one D; 0: each into its own columns
};

template <int MODE, int CHAIN>
__global__ void __launch_bounds__(320) rate_kernel(Args a, long long* out, int* status) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  __shared__ uint32_t tmem_base;
  __shared__ __align__(8) unsigned long long bars[2];
  __shared__ volatile int abort_flag;
  __shared__ volatile int stop;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    abort_flag = 0; stop = 0;
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = threadIdx.x; i < 160 * 1024 / 4; i += blockDim.x) {
    uint32_t x = (uint32_t)i * 2654435761u + blockIdx.x * 40503u; x ^= x >> 13; x *= 0x5bd1e995u; x ^= x >> 15;
    // two bf16 values in (-2, 2): sign, exponent 0x3f / 0x3e.., random mantissa
    uint32_t lo = (x & 0x807fu) | 0x3f00u | ((x >> 3) & 0x0080u), hi = ((x >> 16) & 0x807fu) | 0x3f00u | ((x >> 19) & 0x0080u);
    reinterpret_cast<uint32_t*>(smem)[i] = a.data ? (lo | (hi << 16)) : 0u;
  }
  fence_async_smem();
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base;
  if (warp >= 2 && warp < 6 && a.data) {
    uint32_t v[32];
    for (int cb = 0; cb < 512; cb += 32) {
#pragma unroll
      for (int i = 0; i < 32; ++i) { uint32_t x = (threadIdx.x * 512 + cb + i) * 2654435761u; x ^= x >> 13; x *= 0x5bd1e995u; v[i] = (x & 0x807f807fu) | 0x3f003f00u; }
      ASPD_TMEM_ST32U(tmem + (((warp & 3) * 32u) << 16) + cb, v, 0);
    }
    tmem_wait_st();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t abuf = smem_u32(smem), bbuf = abuf + 32 * 1024, scratch = abuf + 96 * 1024;   // A 32 KB, B 64 KB, scratch 64 KB
  constexpr uint32_t kHalf = 16384;
  if (warp == 0) {
    const uint32_t bar = smem_u32(&bars[0]);
    const long long t0 = clock64();
    uint32_t ph = 0;
    for (int rep = 0; rep < a.nrep; ++rep) {
      const uint32_t d = tmem + (rep & 1) * 128;
      if (MODE == 6) {
        // one tile of the two-tile kernel, both groups: per group two score halves (SS, N = 64) and two P.V halves (TS, K = 64 keys)
#pragma unroll
        for (int g = 0; g < 2; ++g) {
#pragma unroll
          for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
              tc_mma_lane0(tmem + g * 128 + h * 64, smem_desc(abuf + (ks >> 2) * kHalf + (ks & 3) * 32, 16, 1024),
                           smem_desc(bbuf + h * 16384 + (ks >> 2) * 1024 + (ks & 3) * 32, 16, 2048), instr_desc(64, 0), ks > 0);
#pragma unroll
          for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              tc_mma_ts_lane0(tmem + 256 + g * 128, tmem + g * 128 + h * 64 + ks * 8, smem_desc(bbuf + (4 * h + ks) * 4096, 1024, 2048),
                              instr_desc(128, 1), 1);
        }
      } else {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t acc = CHAIN ? (ks > 0) : 0;
          const uint32_t dd = CHAIN ? d : tmem + ((ks & 1) * 128);
          const uint64_t aq = smem_desc(abuf + (ks >> 2) * kHalf + (ks & 3) * 32, 16, 1024);
          switch (MODE) {
            case 0: tc_mma_lane0(dd, aq, smem_desc(bbuf + (ks >> 2) * 1024 + (ks & 3) * 32, 16, 2048), instr_desc(64, 0), acc); break;
            case 1: tc_mma_lane0(dd, aq, smem_desc(bbuf + (ks >> 2) * 1024 + (ks & 3) * 32, 16, 2048), instr_desc(128, 0), acc); break;
            case 2: tc_mma_lane0(tmem, aq, smem_desc(bbuf + (ks >> 2) * 1024 + (ks & 3) * 32, 16, 2048), instr_desc(256, 0), acc); break;
            case 3: tc_mma_lane0(dd, aq, smem_desc(bbuf + ks * 4096, 1024, 2048), instr_desc(128, 1), acc); break;
            case 4: tc_mma_ts_lane0(dd, tmem + 384 + ks * 8, smem_desc(bbuf + ks * 4096, 1024, 2048), instr_desc(128, 1), acc); break;
            case 5: tc_mma_lane0(dd, aq, smem_desc(bbuf + (ks >> 2) * 1024 + (ks & 3) * 32, 16, 2048), instr_desc(128, 0, 64), acc); break;
          }
        }
      }
    }
    tc_commit_lane0(bar);
    bool ok = mbar_wait(bar, ph, &abort_flag, 400000000LL);
    const long long t1 = clock64();
    if (lane == 0) {
      out[blockIdx.x] = t1 - t0;
      if (!ok) *status = -5;
      stop = 1;
    }
  } else if (warp >= 2 && (a.bg & 1) && warp < 6) {
    // TMEM loads as a softmax group would issue them
    float v[32];
    const uint32_t t = tmem + (((warp & 3) * 32u) << 16) + 256;
    float acc = 0.f;
    while (!stop) {
      ASPD_TMEM_LD32(t, v, 0);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) acc += v[i];
    }
    if (acc == 12345.f) out[0] = 0;
  } else if (warp >= 6 && (a.bg & 2)) {
    // shared-memory traffic: 16-byte stores and loads over the scratch area
    uint4 x = make_uint4(lane, 1, 2, 3);
    uint32_t off = (warp - 6) * 4096 + lane * 16;
    uint32_t sum = 0;
    while (!stop) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(scratch + off + i * 512), "r"(x.x), "r"(x.y), "r"(x.z), "r"(x.w) : "memory");
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        uint4 y;
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(y.x), "=r"(y.y), "=r"(y.z), "=r"(y.w) : "r"(scratch + off + i * 512) : "memory");
        sum += y.x;
      }
    }
    if (sum == 12345u) out[0] = 0;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}

int main(int argc, char** argv) {
  int grid = argc > 1 ? atoi(argv[1]) : 148;
  long long* out; int* status;
  cudaMalloc(&out, 148 * 8); cudaMalloc(&status, 4);
  const char* names[] = {"S half SS M128 N64", "S whole SS M128 N128", "SS M128 N256", "PV SS M128 N128 (B MN-major)", "PV TS M128 N128", "S SS M64 N128", "two-tile kernel, one tile of both groups (48 MMAs)"};
  for (int data = 0; data < 2; ++data)
  for (int bg = 0; bg < 4; bg += 3)
    for (int mode = 0; mode < 7; ++mode)
      for (int chain = 1; chain >= 0; --chain) {
        if (mode == 6 && chain == 0) continue;
        if (mode == 2 && chain == 0) continue;
        if (chain == 0) continue;
        Args a{mode, 512, bg, data, chain};
        cudaMemset(status, 0, 4);
        for (int it = 0; it < 2; ++it) {
#define RK(M, C) if (mode == M && chain == C) { cudaFuncSetAttribute(rate_kernel<M, C>, cudaFuncAttributeMaxDynamicSharedMemorySize, 162 * 1024); rate_kernel<M, C><<<grid, 320, 162 * 1024>>>(a, out, status); }
          RK(0, 0) RK(0, 1) RK(1, 0) RK(1, 1) RK(2, 1) RK(3, 0) RK(3, 1) RK(4, 0) RK(4, 1) RK(5, 0) RK(5, 1) RK(6, 1)
        }
        cudaError_t e = cudaDeviceSynchronize();
        if (e != cudaSuccess) { printf("error %s\n", cudaGetErrorString(e)); return 1; }
        std::vector<long long> h(grid); int st;
        cudaMemcpy(h.data(), out, grid * 8, cudaMemcpyDeviceToHost);
        cudaMemcpy(&st, status, 4, cudaMemcpyDeviceToHost);
        double mean = 0; for (auto x : h) mean += x; mean /= grid;
        const int per = mode == 6 ? 48 : 8;
        printf("data %d bg %d chain %d %-32s cycles/MMA %.1f (per group %.0f) status %d\n", data, bg, chain, names[mode], mean / (512.0 * per), mean / 512.0, st);
      }
  return 0;
}
