// Micro-measurements behind two statements of the design notes, runnable on their own:
//   1. the emulated e4m3 accumulation loop (the kernel's own chain8) is pipe bound at about 3.56 cycles per
//      warp-step, and its parts add up: the packed FMA and the conversions share one pipe;
//   2. the fp64 tensor-core instruction m8n8k4 is bit-identical to four chained fma in ascending k, at the
//      rate of the 8 DFMA per lane it replaces.
// Build and run:  python -m paper_2609_39361_b200.probe
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>
#include "lamp_attn.h"
#include "lamp_fwd_sm100.cuh"

using namespace lamp;

// ---------------------------------------------------------------- 1. accumulation loop
// MODE 0: chain8 as the kernel runs it; 1: packed FMA and loads only; 2: rounding (two conversions, two
// f16 -> f32) on an fp32 add, no packed FMA.
template <int MODE>
__device__ __forceinline__ void loop_variant(const float* qf, const float* kf, float (&acc)[4][16]) {
  if (MODE == 0) { chain8<true, false>(qf, kf, 1.0f, acc); return; }
#pragma unroll 2
  for (int kk = 0; kk < kHalf; ++kk) {
    const float4 qv = *reinterpret_cast<const float4*>(qf + kk * kBM);
    const float q4[4] = {qv.x, qv.y, qv.z, qv.w};
    float kv[16];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float4 v = *reinterpret_cast<const float4*>(kf + kk * kKfStride + 4 * c);
      kv[4 * c] = v.x; kv[4 * c + 1] = v.y; kv[4 * c + 2] = v.z; kv[4 * c + 3] = v.w;
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      uint64_t qq;
      asm("mov.b64 %0, {%1, %1};" : "=l"(qq) : "f"(q4[a]));
#pragma unroll
      for (int b = 0; b < 16; b += 2) {
        float t0, t1;
        if (MODE == 1) {
          fma_x2(t0, t1, kv[b], kv[b + 1], qq, acc[a][b], acc[a][b + 1]);
        } else {
          t0 = acc[a][b] + kv[b]; t1 = acc[a][b + 1];
          rne_e4m3_x2(t0, t1);
        }
        acc[a][b] = t0; acc[a][b + 1] = t1;
      }
    }
  }
}
template <int MODE, int W>
__global__ void __launch_bounds__(128 * W, 1) loop_kernel(float* out, int reps, long long* cyc) {
  extern __shared__ unsigned char smem[];
  float* qs = reinterpret_cast<float*>(smem);     // [128 kk][128 rows]
  float* kfa = qs + kHalf * kBM;                  // [128 kk][kKfStride]
  for (int i = threadIdx.x; i < kHalf * kBM; i += blockDim.x) qs[i] = 0.01f * ((i * 37) % 101 - 50);
  for (int i = threadIdx.x; i < kHalf * kKfStride; i += blockDim.x) kfa[i] = 0.02f * ((i * 53) % 89 - 44);
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float acc[4][16];
  for (int a = 0; a < 4; ++a) for (int b = 0; b < 16; ++b) acc[a][b] = 0.0f;
  const long long t0 = clock64();
  for (int r = 0; r < reps; ++r)
    loop_variant<MODE>(qs + (warp & 3) * 32 + 4 * (lane >> 2), kfa + kf_pos(16 * (lane & 3)), acc);
  const long long t1 = clock64();
  float s = 0;
  for (int a = 0; a < 4; ++a) for (int b = 0; b < 16; ++b) s += acc[a][b];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
  if (threadIdx.x == 0 && blockIdx.x == 0) *cyc = t1 - t0;
}
template <int MODE, int W>
static void run_loop(float* o, long long* c, const char* what) {
  const int smem = (kHalf * kBM + kHalf * kKfStride) * 4, reps = 32;
  cudaFuncSetAttribute(loop_kernel<MODE, W>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  for (int it = 0; it < 2; ++it) { loop_kernel<MODE, W><<<148, 128 * W, smem>>>(o, reps, c); cudaDeviceSynchronize(); }
  long long hc = 0;
  cudaMemcpy(&hc, c, 8, cudaMemcpyDeviceToHost);
  printf("  %-52s %d warps per scheduler: %.3f cycles per warp-step  (%s)\n", what, W,
         (double)hc / reps / kHalf / 64 / W, cudaGetErrorString(cudaGetLastError()));
}

// ---------------------------------------------------------------- 2. fp64 tensor-core instruction
__global__ void dmma_check(const double* A, const double* B, const double* C, double* D) {   // A[8][4], B[4][8], C[8][8]
  const int l = threadIdx.x, g = l >> 2, t = l & 3;
  double c0 = C[g * 8 + 2 * t], c1 = C[g * 8 + 2 * t + 1];
  dmma_884(c0, c1, A[g * 4 + t], B[t * 8 + g]);
  D[g * 8 + 2 * t] = c0; D[g * 8 + 2 * t + 1] = c1;
}
template <bool TENSOR>
__global__ void fp64_rate(double* out, int reps, long long* cyc) {
  const int l = threadIdx.x;
  double c[16];
  for (int i = 0; i < 16; ++i) c[i] = l * 0.001 + i;
  const double a = 1.0 + l * 1e-9, b = 1.0 - l * 1e-9;
  __syncthreads();
  const long long t0 = clock64();
  for (int r = 0; r < reps; ++r) {
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
      if (TENSOR) dmma_884(c[i], c[i + 1], a, b);
      else { c[i] = fma(a, b, c[i]); c[i + 1] = fma(a, b, c[i + 1]); }
    }
  }
  const long long t1 = clock64();
  double s = 0;
  for (int i = 0; i < 16; ++i) s += c[i];
  out[blockIdx.x * blockDim.x + l] = s;
  if (l == 0 && blockIdx.x == 0) *cyc = t1 - t0;
}

int main() {
  float* o; long long* c;
  cudaMalloc(&o, 148 * 1024 * 8); cudaMalloc(&c, 8);
  printf("1. emulated e4m3 accumulation loop (one warp-step = one channel of one (query, key) pair for 32 lanes)\n");
  run_loop<0, 1>(o, c, "the kernel's loop");
  run_loop<0, 2>(o, c, "the kernel's loop");
  run_loop<0, 4>(o, c, "the kernel's loop");
  run_loop<1, 2>(o, c, "packed FMA and operand loads only");
  run_loop<2, 2>(o, c, "rounding only (2 conversions, 2 f16->f32, on an add)");

  printf("2. mma.sync.m8n8k4.f64 against fma chains (operand exponents spread over 2^60)\n");
  double hA[32], hB[32], hC[64], hD[64], *A, *B, *C, *D;
  cudaMalloc(&A, 256); cudaMalloc(&B, 256); cudaMalloc(&C, 512); cudaMalloc(&D, 512);
  srand(1);
  long long n = 0, bad_fwd = 0, bad_rev = 0;
  for (int trial = 0; trial < 2000; ++trial) {
    for (int i = 0; i < 32; ++i) {
      hA[i] = ldexp((rand() / (double)RAND_MAX) * 2 - 1, rand() % 60 - 30);
      hB[i] = ldexp((rand() / (double)RAND_MAX) * 2 - 1, rand() % 60 - 30);
    }
    for (int i = 0; i < 64; ++i) hC[i] = ldexp((rand() / (double)RAND_MAX) * 2 - 1, rand() % 60 - 30);
    cudaMemcpy(A, hA, 256, cudaMemcpyHostToDevice); cudaMemcpy(B, hB, 256, cudaMemcpyHostToDevice);
    cudaMemcpy(C, hC, 512, cudaMemcpyHostToDevice);
    dmma_check<<<1, 32>>>(A, B, C, D);
    cudaMemcpy(hD, D, 512, cudaMemcpyDeviceToHost);
    for (int m = 0; m < 8; ++m)
      for (int nn = 0; nn < 8; ++nn) {
        double f = hC[m * 8 + nn], r = hC[m * 8 + nn];
        for (int k = 0; k < 4; ++k) f = fma(hA[m * 4 + k], hB[k * 8 + nn], f);
        for (int k = 3; k >= 0; --k) r = fma(hA[m * 4 + k], hB[k * 8 + nn], r);
        bad_fwd += f != hD[m * 8 + nn]; bad_rev += r != hD[m * 8 + nn]; ++n;
      }
  }
  printf("  %lld elements: %lld differ from the fma chain k = 0..3, %lld from the chain k = 3..0  (%s)\n", n, bad_fwd,
         bad_rev, cudaGetErrorString(cudaGetLastError()));
  for (int w = 1; w <= 2; ++w) {
    long long hc = 0;
    for (int it = 0; it < 2; ++it) { fp64_rate<true><<<148, 128 * w>>>((double*)o, 4096, c); cudaDeviceSynchronize(); }
    cudaMemcpy(&hc, c, 8, cudaMemcpyDeviceToHost);
    printf("  %d warps per scheduler: %.2f cycles per m8n8k4 instruction", w, (double)hc / 4096 / 8 / w);
    for (int it = 0; it < 2; ++it) { fp64_rate<false><<<148, 128 * w>>>((double*)o, 4096, c); cudaDeviceSynchronize(); }
    cudaMemcpy(&hc, c, 8, cudaMemcpyDeviceToHost);
    printf(", %.2f per DFMA\n", (double)hc / 4096 / 16 / w);
  }
  return bad_fwd != 0;
}
