// Stand-alone probe of the FP64 fused multiply-add issue rate on the current GPU,
// the unit that bounds the direct scoring kernel.  Two kernels of independent fma
// chains (round toward minus infinity, as the scoring kernels use), one block of
// 16 warps per SM:
//
//   registers : all three sources of every fma are ordinary per-lane registers;
//   uniform   : one source is a warp-uniform constant that the compiler keeps in a
//               uniform register for the whole loop -- the form the direct scoring
//               kernel's fmas have (demand operand uniform, candidate constant,
//               accumulator);
//   shared    : three register sources again, but runs of consecutive fmas have one
//               source register in common (the operand-reuse case).
//
// Output: one JSON line with the rates in warp-instructions per clock per SM
// (cycles from clock64 of the slowest block), the SM count and the clock seen.
// A measurement aid of bench.py (bench.py --fp64-probe runs it); the library does not use it.
#include <cstdint>
#include <cstdio>
#include <cuda_runtime.h>

namespace {

constexpr int kChains = 4;        // independent accumulators per thread
constexpr int kUnroll = 8;        // fma groups per loop trip
constexpr int kWarps = 16;        // warps per block, one block per SM
__constant__ double c_u[kChains * kUnroll];

template <int MODE>
__global__ void __launch_bounds__(kWarps * 32, 1)
fma_rate_kernel(const double* __restrict__ in, double* __restrict__ out, int trips, long long* __restrict__ cycles) {
  double x[kChains], y[kChains], acc[kChains];
#pragma unroll
  for (int c = 0; c < kChains; ++c) {
    x[c] = in[threadIdx.x + 32 * c];
    y[c] = in[threadIdx.x + 32 * (c + kChains)];
    acc[c] = in[c] + 6755399441055744.0;
  }
  const long long t0 = clock64();
  for (int t = 0; t < trips; ++t) {
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
#pragma unroll
      for (int c = 0; c < kChains; ++c)
        acc[c] = MODE == 1 ? __fma_rd(c_u[u * kChains + c], y[c], acc[c])
                 : MODE == 2 ? __fma_rd(x[u % kChains], y[c], acc[c])
                             : __fma_rd(x[(c + u) % kChains], y[c], acc[c]);
  }
  const long long t1 = clock64();
  double s = 0.0;
#pragma unroll
  for (int c = 0; c < kChains; ++c) s += acc[c];
  out[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

template <int MODE>
bool measure(int n_sms, const double* d_in, double* d_out, long long* d_cycles, double* rate, double* mhz) {
  const int trips = 4000;
  cudaEvent_t e0, e1;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return false;
  for (int rep = 0; rep < 4; ++rep) {          // the first launches also bring the clock up
    cudaEventRecord(e0);
    fma_rate_kernel<MODE><<<n_sms, kWarps * 32>>>(d_in, d_out, trips, d_cycles);
    cudaEventRecord(e1);
    if (cudaEventSynchronize(e1) != cudaSuccess) return false;
  }
  float ms = 0.f;
  cudaEventElapsedTime(&ms, e0, e1);
  long long* h = new long long[n_sms];
  cudaMemcpy(h, d_cycles, sizeof(long long) * n_sms, cudaMemcpyDeviceToHost);
  long long worst = 0;
  for (int b = 0; b < n_sms; ++b) worst = h[b] > worst ? h[b] : worst;
  delete[] h;
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (worst <= 0 || cudaGetLastError() != cudaSuccess) return false;
  *rate = (double)trips * kUnroll * kChains * kWarps / (double)worst;
  *mhz = (double)worst / (ms * 1e3);
  return true;
}

}  // namespace

int main() {
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, 0) != cudaSuccess) { std::printf("{\"error\": \"no CUDA device\"}\n"); return 1; }
  const int n_sms = prop.multiProcessorCount;
  double *d_in = nullptr, *d_out = nullptr;
  long long* d_cycles = nullptr;
  if (cudaMalloc(&d_in, 4096 * sizeof(double)) != cudaSuccess ||
      cudaMalloc(&d_out, (size_t)n_sms * kWarps * 32 * sizeof(double)) != cudaSuccess ||
      cudaMalloc(&d_cycles, sizeof(long long) * n_sms) != cudaSuccess) {
    std::printf("{\"error\": \"allocation failed\"}\n");
    return 1;
  }
  double h_in[4096];
  for (int i = 0; i < 4096; ++i) h_in[i] = 1e-7 * (i % 977 + 1);
  cudaMemcpy(d_in, h_in, sizeof(h_in), cudaMemcpyHostToDevice);
  double h_u[kChains * kUnroll];
  for (int i = 0; i < kChains * kUnroll; ++i) h_u[i] = 1000.0 + i;
  cudaMemcpyToSymbol(c_u, h_u, sizeof(h_u));
  double r_reg = 0, r_uni = 0, r_shr = 0, mhz_reg = 0, mhz_uni = 0, mhz_shr = 0;
  const bool ok = measure<0>(n_sms, d_in, d_out, d_cycles, &r_reg, &mhz_reg) &&
                  measure<1>(n_sms, d_in, d_out, d_cycles, &r_uni, &mhz_uni) &&
                  measure<2>(n_sms, d_in, d_out, d_cycles, &r_shr, &mhz_shr);
  cudaFree(d_in); cudaFree(d_out); cudaFree(d_cycles);
  if (!ok) { std::printf("{\"error\": \"launch failed\"}\n"); return 1; }
  std::printf("{\"gpu\": \"%s\", \"sms\": %d, \"fma_warp_inst_per_clk_per_sm\": {\"register_sources\": %.4f, "
              "\"one_uniform_source\": %.4f, \"register_sources_one_shared\": %.4f}, "
              "\"sm_mhz_seen\": {\"register_sources\": %.0f, \"one_uniform_source\": %.0f, \"register_sources_one_shared\": %.0f}}\n",
              prop.name, n_sms, r_reg, r_uni, r_shr, mhz_reg, mhz_uni, mhz_shr);
  return 0;
}
