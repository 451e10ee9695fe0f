// Small kernels around the layer.
//   residual stream between the layers of a decode-step loop: h_out = round_to_storage(h_in + y), where y is a
//     layer's fp32 output and h the hidden states in the layers' storage type; the add is one fp32 operation and the
//     rounding to bf16 is round-to-nearest-even, so the next layer's input is a defined bit pattern;
//   bf16 output type: the fp32 sum of the layer rounded once, after the last addition;
//   self-test of the bounded device-side wait (failure detection without hanging anything).
#include <algorithm>
#include <cuda_bf16.h>

#include "tc_ptx.cuh"

namespace pcomoe {
namespace {

__global__ void __launch_bounds__(256) residual_cast_bf16_kernel(const uint4 *h_in, const float4 *y, uint4 *h_out,
                                                                 int64_t n8, const __nv_bfloat16 *h_in_s,
                                                                 const float *y_s, __nv_bfloat16 *h_out_s,
                                                                 int64_t n) {
  pdl_grid_wait();
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += stride) {
    const uint4 hv = h_in[i];
    const float4 a = y[2 * i], b = y[2 * i + 1];
    const __nv_bfloat162 *hp = reinterpret_cast<const __nv_bfloat162 *>(&hv);
    const float ys[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint4 ov;
    __nv_bfloat162 *op = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float2 f = __bfloat1622float2(hp[k]);
      op[k] = __floats2bfloat162_rn(__fadd_rn(f.x, ys[2 * k]), __fadd_rn(f.y, ys[2 * k + 1]));
    }
    h_out[i] = ov;
  }
  // tail that does not fill a vector of eight
  for (int64_t i = 8 * n8 + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
    h_out_s[i] = __float2bfloat16_rn(__fadd_rn(__bfloat162float(h_in_s[i]), y_s[i]));
}

__global__ void __launch_bounds__(256) residual_cast_f32_kernel(const float *h_in, const float *y, float *h_out, int64_t n) {
  pdl_grid_wait();
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) h_out[i] = __fadd_rn(h_in[i], y[i]);
}

// y in the layer's bf16 output type: the fp32 accumulator rounded once, to nearest-even, after the last addition.
__global__ void __launch_bounds__(256) cast_y_bf16_kernel(const float4 *acc, uint4 *out, int64_t n8, const float *acc_s,
                                                          __nv_bfloat16 *out_s, int64_t n) {
  pdl_grid_wait();
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += stride) {
    const float4 a = __ldcs(acc + 2 * i), b = __ldcs(acc + 2 * i + 1);
    uint4 ov;
    __nv_bfloat162 *op = reinterpret_cast<__nv_bfloat162 *>(&ov);
    op[0] = __floats2bfloat162_rn(a.x, a.y);
    op[1] = __floats2bfloat162_rn(a.z, a.w);
    op[2] = __floats2bfloat162_rn(b.x, b.y);
    op[3] = __floats2bfloat162_rn(b.z, b.w);
    out[i] = ov;
  }
  for (int64_t i = 8 * n8 + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
    out_s[i] = __float2bfloat16_rn(acc_s[i]);
}

// Self-test of the bounded wait: one warp waits, with the same helper and limit as the GEMM kernels, on an
// mbarrier that nothing will ever arrive on (no copy, MMA or other CTA is involved), and then takes the same
// give-up path: the status word receives PCOMOE_ERR_TIMEOUT and the kernel returns.
__global__ void __launch_bounds__(32) wait_probe_kernel(int32_t *status_word, uint64_t limit_ns) {
  pdl_grid_wait();
  __shared__ __align__(8) uint64_t s_bar;
  __shared__ int s_abort;
  if (threadIdx.x == 0) {
    s_abort = 0;
    mbar_init(smem_u32(&s_bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  bool done = true;
  if (threadIdx.x == 0) done = mbar_wait(smem_u32(&s_bar), 0, &s_abort, limit_ns);
  __syncwarp();
  if (s_abort) timeout_record_and_drain(status_word);
  (void)done;
}

}  // namespace

pcomoe_status launch_cast_y(const pcomoe_layer *L, int32_t T, const float *y_acc, void *y_out, cudaStream_t st) {
  const int64_t n = (int64_t)T * L->cfg.hidden;
  const bool vec = (((uintptr_t)y_acc | (uintptr_t)y_out) & 15) == 0;
  const int64_t n8 = vec ? n / 8 : 0;
  const int grid = (int)std::min<int64_t>((n / 8 + 255) / 256 + 1, (int64_t)L->sm_count * 8);
  PCOMOE_CUDA_TRY(launch_pdl(cast_y_bf16_kernel, dim3(grid), dim3(256), 0, st, (const float4 *)y_acc, (uint4 *)y_out, n8,
                             y_acc, (__nv_bfloat16 *)y_out, n));
  count_launch();
  return PCOMOE_OK;
}

pcomoe_status launch_wait_probe(int32_t *status_word, cudaStream_t st) {
  PCOMOE_CUDA_TRY(launch_pdl(wait_probe_kernel, dim3(1), dim3(32), 0, st, status_word, wait_limit_ns()));
  count_launch();
  return PCOMOE_OK;
}

pcomoe_status launch_residual_cast(const pcomoe_layer *L, int32_t T, const void *h_in, const float *y, void *h_out,
                                   cudaStream_t st) {
  const int64_t n = (int64_t)T * L->cfg.hidden;
  int grid = (int)std::min<int64_t>((n / 8 + 255) / 256 + 1, (int64_t)L->sm_count * 8);
  if (L->cfg.in_dtype == PCOMOE_BF16) {
    const bool vec = (((uintptr_t)h_in | (uintptr_t)h_out | (uintptr_t)y) & 15) == 0;
    const int64_t n8 = vec ? n / 8 : 0;
    PCOMOE_CUDA_TRY(launch_pdl(residual_cast_bf16_kernel, dim3(grid), dim3(256), 0, st, (const uint4 *)h_in,
                               (const float4 *)y, (uint4 *)h_out, n8, (const __nv_bfloat16 *)h_in, y,
                               (__nv_bfloat16 *)h_out, n));
  } else {
    PCOMOE_CUDA_TRY(launch_pdl(residual_cast_f32_kernel, dim3(grid), dim3(256), 0, st, (const float *)h_in, y,
                               (float *)h_out, n));
  }
  count_launch();
  return PCOMOE_OK;
}

}  // namespace pcomoe
