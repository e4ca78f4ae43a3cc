// Probe behind the integer roof of the race kernel: how many clocks does a warp instruction of each
// kind cost one SM sub-partition, and do wide multiplies, three-input xors and FP32 FMAs overlap?
// Every thread runs independent chains (opaque inline PTX, so nothing is folded); 148 blocks, one
// per SM; the figure printed is clocks per loop iteration per warp on its sub-partition at the
// nominal 1965 MHz.  Philox4x32-10 is exactly this mix: per round two wide multiplies, each
// followed by a dependent three-input xor.
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdint.h>
#define ITERS 4096
__device__ __forceinline__ uint32_t xor3(uint32_t a, uint32_t b, uint32_t c) { uint32_t d; asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(d) : "r"(a), "r"(b), "r"(c)); return d; }
__device__ __forceinline__ void mulwide(uint32_t a, uint32_t m, uint32_t& hi, uint32_t& lo) { asm("{.reg .u64 t; mul.wide.u32 t, %2, %3; mov.b64 {%1,%0}, t;}" : "=r"(hi), "=r"(lo) : "r"(a), "r"(m)); }
template <int NW, int NL, int NF, int THREADS>
__global__ void __launch_bounds__(THREADS) k(uint32_t* out, uint32_t seed) {
  uint32_t a[8], al[8], b[8]; float f[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) { a[j] = seed + threadIdx.x * 8 + j; al[j] = 0; b[j] = a[j] * 3u; f[j] = (float)j; }
  const uint32_t k1 = seed * 7u, k2 = seed * 11u;
  for (int it = 0; it < ITERS; ++it) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (j < NW) { uint32_t hi, lo; mulwide(a[j], 0xD2511F53u, hi, lo); a[j] = hi; al[j] = lo; }
      if (j < NL) b[j] = xor3(b[j], k1, k2);
      if (j < NF) f[j] = fmaf(f[j], 1.0001f, 0.5f);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) if (j < NW) a[j] = xor3(a[j], al[j], k1) ;   // like Philox: one LOP3 per product, dependent
  }
  uint32_t acc = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) acc ^= a[j] ^ b[j] ^ __float_as_uint(f[j]);
  if (acc == 0x12345678u) out[0] = acc;
}
template <int NW, int NL, int NF, int THREADS> void run(uint32_t* d) {
  cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  k<NW, NL, NF, THREADS><<<148, THREADS>>>(d, 12345u);
  cudaEventRecord(e0);
  k<NW, NL, NF, THREADS><<<148, THREADS>>>(d, 12345u);
  cudaEventRecord(e1); cudaEventSynchronize(e1);
  float ms; cudaEventElapsedTime(&ms, e0, e1);
  double cyc = ms * 1e-3 * 1.965e9 / ITERS / (THREADS / 128.0);   // cycles per iteration per warp on its SMSP
  printf("threads %4d: wide %d (+%d dependent lop3)  extra lop3 %d  ffma %d : %6.2f cycles per warp-iteration  (%d instrs)\n", THREADS, NW, NW, NL, NF, cyc, 2 * NW + NL + NF);
}
int main() {
  uint32_t* d; cudaMalloc(&d, 64);
  run<4,0,0,1024>(d); run<8,0,0,1024>(d); run<0,8,0,1024>(d); run<0,0,8,1024>(d);
  run<4,4,0,1024>(d); run<4,8,0,1024>(d); run<4,0,8,1024>(d); run<4,4,8,1024>(d); run<4,8,8,1024>(d);
  run<4,4,0,512>(d); run<4,8,8,512>(d); run<4,4,0,256>(d); run<4,8,8,256>(d);
  return 0;
}
