// Machine peaks measured in place, for benchmarks: the rates that bound the ALU-bound goodput
// sweep (fp32 FMA lanes, special-function unit) and the read-only streaming fitness kernel, at
// the clocks the GPU runs at when the benchmark does.  Not part of the method.
#include "common.cuh"

namespace {

constexpr int PROBE_THREADS = 256;
constexpr int FMA_CHAINS = 8;     // independent accumulators per thread: hides the FMA latency
constexpr int MUFU_CHAINS = 4;

__global__ void __launch_bounds__(PROBE_THREADS) fma_chain_kernel(int iters, float a, float b, float *out) {
  float x[FMA_CHAINS];
#pragma unroll
  for (int k = 0; k < FMA_CHAINS; ++k) x[k] = (float)(threadIdx.x + k);
  for (int i = 0; i < iters; ++i) {
#pragma unroll
    for (int k = 0; k < FMA_CHAINS; ++k) x[k] = fmaf(x[k], a, b);
  }
  float s = 0.f;
#pragma unroll
  for (int k = 0; k < FMA_CHAINS; ++k) s += x[k];
  if (s == 123.456f) out[0] = s;          // keeps the chains alive; practically never true
}

__global__ void __launch_bounds__(PROBE_THREADS) mufu_chain_kernel(int iters, float *out) {
  float x[MUFU_CHAINS];
#pragma unroll
  for (int k = 0; k < MUFU_CHAINS; ++k) x[k] = 1.5f + (float)((threadIdx.x + k) & 7);
  for (int i = 0; i < iters; ++i) {
#pragma unroll
    for (int k = 0; k < MUFU_CHAINS; ++k) {   // ex2(lg2(x)) = x: two special-function ops, the value stays put
      float y;
      asm volatile("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x[k]));
      asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(x[k]) : "f"(y));
    }
  }
  float s = 0.f;
#pragma unroll
  for (int k = 0; k < MUFU_CHAINS; ++k) s += x[k];
  if (s == -1.f) out[0] = s;
}

// read-only stream: every thread sums the 16-byte pieces it is dealt, several loads in flight
__global__ void __launch_bounds__(PROBE_THREADS) read_stream_kernel(const uint4 *__restrict__ src, size_t n, uint32_t *out) {
  uint32_t acc = 0;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (; i + 3 * stride < n; i += 4 * stride) {
    uint4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                   : "=r"(v[k].x), "=r"(v[k].y), "=r"(v[k].z), "=r"(v[k].w) : "l"(src + i + k * stride));
#pragma unroll
    for (int k = 0; k < 4; ++k) acc ^= v[k].x ^ v[k].y ^ v[k].z ^ v[k].w;
  }
  for (; i < n; i += stride) {
    const uint4 v = __ldg(src + i);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
  if (acc == 0x9E3779B9u) out[0] = acc;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

int sched_measure_peaks(sched_ctx *ctx, const void *d_buffer, uint64_t bytes, int32_t reps, double *h_fp32_lane_ops_per_s,
                        double *h_mufu_ops_per_s, double *h_read_bytes_per_s) {
  if (!ctx) { set_error(nullptr, "sched_measure_peaks: ctx is NULL"); return SCHED_ERR_INVALID_ARG; }
  if (reps < 1 || !h_fp32_lane_ops_per_s || !h_mufu_ops_per_s || !h_read_bytes_per_s ||
      (d_buffer && (((uintptr_t)d_buffer & 15) != 0))) {
    set_error(ctx, "sched_measure_peaks: reps >= 1, non-NULL outputs, a 16-byte aligned buffer");
    return SCHED_ERR_INVALID_ARG;
  }
  cudaEvent_t e0, e1;
  SCHED_CUDA_CHECK(ctx, cudaEventCreate(&e0));
  SCHED_CUDA_CHECK(ctx, cudaEventCreate(&e1));
  float *d_out = (float *)ctx->d_best_idx;     // a word of context scratch the kernels practically never write
  const int blocks = ctx->num_sms * 8;
  const int fma_iters = 1 << 14, mufu_iters = 1 << 12;
  auto timed = [&](auto launch, double &seconds) -> int {
    launch();                                                     // warm-up
    SCHED_CUDA_CHECK(ctx, cudaEventRecord(e0, ctx->stream));
    for (int r = 0; r < reps; ++r) launch();
    SCHED_CUDA_CHECK(ctx, cudaEventRecord(e1, ctx->stream));
    SCHED_CUDA_CHECK(ctx, cudaEventSynchronize(e1));
    float ms = 0.f;
    SCHED_CUDA_CHECK(ctx, cudaEventElapsedTime(&ms, e0, e1));
    SCHED_CUDA_CHECK(ctx, cudaGetLastError());
    ctx->launches += reps + 1;
    seconds = (double)ms * 1e-3 / reps;
    return SCHED_OK;
  };
  double t = 0.0;
  int rc = timed([&] { fma_chain_kernel<<<blocks, PROBE_THREADS, 0, ctx->stream>>>(fma_iters, 0.999f, 0.001f, d_out); }, t);
  if (rc != SCHED_OK) return rc;
  *h_fp32_lane_ops_per_s = (double)blocks * PROBE_THREADS * FMA_CHAINS * fma_iters / t;
  rc = timed([&] { mufu_chain_kernel<<<blocks, PROBE_THREADS, 0, ctx->stream>>>(mufu_iters, d_out); }, t);
  if (rc != SCHED_OK) return rc;
  *h_mufu_ops_per_s = (double)blocks * PROBE_THREADS * MUFU_CHAINS * 2.0 * mufu_iters / t;
  *h_read_bytes_per_s = 0.0;
  if (d_buffer && bytes >= 16) {
    const size_t n = (size_t)(bytes / 16);
    rc = timed([&] { read_stream_kernel<<<ctx->num_sms * 16, PROBE_THREADS, 0, ctx->stream>>>((const uint4 *)d_buffer, n, (uint32_t *)d_out); }, t);
    if (rc != SCHED_OK) return rc;
    *h_read_bytes_per_s = (double)n * 16.0 / t;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  return SCHED_OK;
}

#pragma GCC visibility pop
}  // extern "C"
