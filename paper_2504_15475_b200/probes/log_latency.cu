// Latency of the pieces of the deciding logarithm (csrc/ersd_math.cuh): one warp alone on an SM,
// dependent chains, SM clocks per call.  Needs -I <package>/csrc.
#include <cuda_runtime.h>
#include <cstdio>
#include "ersd_math.cuh"
using namespace ersd;
__global__ void k(long long* out, double* sink, uint32_t x0) {
  const int n = 64;
  uint32_t x = x0 + threadIdx.x;
  double acc = 0.0;
  long long t0 = clock64();
  for (int i = 0; i < n; ++i) { acc += exact_ln_e(x); x = x * 1664525u + 1013904223u + (uint32_t)(acc > 1e300); }
  long long t1 = clock64();
  double d = 1.5 + threadIdx.x * 1e-3;
  for (int i = 0; i < n; ++i) d = 1.0 + recip_1_4(d) ;   // in [1, 4]
  long long t2 = clock64();
  double s = 0.01 + threadIdx.x * 1e-4;
  for (int i = 0; i < n; ++i) s = 0.01 + atanh_tail<16>(s) * 1e-3;
  long long t3 = clock64();
  double u = 0.3 + threadIdx.x * 1e-3;
  for (int i = 0; i < n; ++i) u = 0.3 + fabs(ln_pos(u)) * 0.1;
  long long t4 = clock64();
  double f = 1.0 + threadIdx.x * 1e-3;
  for (int i = 0; i < n * 8; ++i) f = fma(f, 0.999, 0.001);
  long long t5 = clock64();
  if (threadIdx.x == 0) { out[0] = (t1 - t0) / n; out[1] = (t2 - t1) / n; out[2] = (t3 - t2) / n; out[3] = (t4 - t3) / n; out[4] = (t5 - t4) / (n * 8); }
  sink[threadIdx.x] = acc + d + s + u + f;
}
int main() {
  long long* out; double* sink; cudaMalloc(&out, 64); cudaMalloc(&sink, 32 * 8);
  for (int rep = 0; rep < 2; ++rep) k<<<1, 32>>>(out, sink, 12345u);
  long long h[5]; cudaMemcpy(h, out, 40, cudaMemcpyDeviceToHost);
  printf("clocks per call, one warp alone: exact_ln_e %lld, recip_1_4 %lld, atanh_tail<16> %lld, ln_pos %lld, one dependent DFMA %lld\n", h[0], h[1], h[2], h[3], h[4]);
  return cudaGetLastError() != cudaSuccess;
}
