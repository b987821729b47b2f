// Probe (development aid, not part of the library): throughput per SM sub-partition of the instructions the
// exponent passes are made of: ex2 (mode 1; with an add: 0), FFMA (2), the bf16 pair conversion (3), packed
// FFMA2 / FADD2 (4 / 5; 8 instructions per 16 counted), two ex2 per conversion (6).  8 warps per SM.
#include <cstdio>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
__device__ __forceinline__ float ex2(float x) { float y; asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
template <int MODE>
__global__ void k(float* out, long long* cyc, int n) {
  float x[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) x[i] = -0.001f * (threadIdx.x + i);
  __syncthreads();
  long long t0 = clock64();
  for (int it = 0; it < n; ++it) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if (MODE == 0) x[i] = ex2(x[i]) - 1.0f;             // 1 MUFU + 1 FADD per element
      if (MODE == 1) x[i] = ex2(x[i]);                     // MUFU only
      if (MODE == 2) x[i] = fmaf(x[i], 0.999f, -0.001f);   // FMA only
      if (MODE == 3) { __nv_bfloat162 h = __floats2bfloat162_rn(x[i], x[i ^ 1]); x[i] = __uint_as_float(*reinterpret_cast<unsigned*>(&h)) ; }  // pack
      if (MODE == 4 && (i & 1) == 0) { float2 r = __ffma2_rn(make_float2(x[i], x[i + 1]), make_float2(0.999f, 0.999f), make_float2(-0.001f, -0.001f)); x[i] = r.x; x[i + 1] = r.y; }
      if (MODE == 5 && (i & 1) == 0) { float2 r = __fadd2_rn(make_float2(x[i], x[i + 1]), make_float2(-0.001f, -0.001f)); x[i] = r.x; x[i + 1] = r.y; }
      if (MODE == 6) { x[i] = ex2(x[i]); if ((i & 1) == 0) { __nv_bfloat162 h = __floats2bfloat162_rn(x[i], x[i + 1]); x[i + 1] += __uint_as_float(*reinterpret_cast<unsigned*>(&h)); } }   // 2 MUFU : 1 pack
    }
  }
  long long t1 = clock64();
  float s = 0; for (int i = 0; i < 16; ++i) s += x[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
  if (threadIdx.x == 0) cyc[blockIdx.x] = t1 - t0;
}
int main() {
  float* out; long long* cyc; cudaMalloc(&out, 148 * 1024 * 4); cudaMalloc(&cyc, 148 * 8);
  for (int warps = 8; warps <= 8; warps *= 2)
    for (int mode = 0; mode < 7; ++mode) {
      const int n = 2000;
      for (int r = 0; r < 2; ++r) {
        if (mode == 0) k<0><<<148, warps * 32>>>(out, cyc, n);
        if (mode == 1) k<1><<<148, warps * 32>>>(out, cyc, n);
        if (mode == 2) k<2><<<148, warps * 32>>>(out, cyc, n);
        if (mode == 3) k<3><<<148, warps * 32>>>(out, cyc, n);
        if (mode == 4) k<4><<<148, warps * 32>>>(out, cyc, n);
        if (mode == 5) k<5><<<148, warps * 32>>>(out, cyc, n);
        if (mode == 6) k<6><<<148, warps * 32>>>(out, cyc, n);
      }
      cudaDeviceSynchronize();
      long long h[148]; cudaMemcpy(h, cyc, sizeof(h), cudaMemcpyDeviceToHost);
      double c = h[0];
      // per SMSP: warps/4 warps, each n*16 instructions of the kind
      printf("warps/SM %2d mode %d: %.2f cycles per warp-instruction per SMSP (%.1f lanes/clk/SM)\n", warps, mode, c / (n * 16.0 * warps / 4), 32.0 * 4 / (c / (n * 16.0 * warps / 4)));
    }
  return 0;
}
