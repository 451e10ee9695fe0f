// Plain-FMA kernels for the two stages of the layer.  They cover every size and both storage
// types (the fp32 layer runs here; bf16 layers whose sizes the tensor-core kernels do not take
// run here too).  One block per row; a warp per output element, lanes along the contraction.
//   stage 1: U[r,:] = SiLU(W_gate^(i) h_t) (.) (W_up^(i) h_t)            (Sec. 4.1, U_e)
//   stage 2: y[token,:] += w * W_down^(j) U[row,:]                        (Sec. 4.1, D_e; Sec. 4.3 sum)
#include "common.cuh"

namespace pcomoe {

template <typename E> __device__ __forceinline__ float to_f(E v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename E> __device__ __forceinline__ E from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

// group of a row: the g with offsets[g] <= row < offsets[g+1]; -1 when row is past the end
__device__ __forceinline__ int find_group(const int32_t *offsets, int n, int row) {
  if (row >= offsets[n]) return -1;
  int g = 0;
  while (g + 1 < n && offsets[g + 1] <= row) ++g;
  return g;
}

struct SimtArgs {
  const int32_t *offsets;   // [G+1] rows per group, or NULL: one group, `rows` rows
  const int32_t *row_src;   // stage 1: token of a row; stage 2: intermediate row of a row (NULL: identity)
  const int32_t *row_token; // stage 2: token of a row (NULL: identity)
  const float *row_w;       // stage 2: weight of a row (NULL: 1)
  int32_t G, rows, H, F;    // F = contraction / output width of this call (F or F_sh)
  int32_t limit_src;        // bound of row_src values (T in stage 1, row capacity of U in stage 2)
  int32_t T;
  DevPlan *plan;
};

template <typename E>
__global__ void __launch_bounds__(128) simt_stage1_kernel(const SimtArgs a, const E *h, const E *wg,
                                                          const E *wu, E *U) {
  extern __shared__ float hs[];
  __shared__ int sg, stok;
  const int row = blockIdx.x;
  if (threadIdx.x == 0) {
    sg = a.offsets ? find_group(a.offsets, a.G, row) : (row < a.rows ? 0 : -1);
    int tok = sg < 0 ? 0 : (a.row_src ? a.row_src[row] : row);
    if ((unsigned)tok >= (unsigned)a.limit_src) {
      atomicCAS(&a.plan->status, 0, PCOMOE_ERR_INDEX);
      sg = -1;
    }
    stok = tok;
  }
  __syncthreads();
  const int g = sg;
  if (g < 0) return;
  const E *hr = h + (size_t)stok * a.H;
  for (int k = threadIdx.x; k < a.H; k += blockDim.x) hs[k] = to_f<E>(hr[k]);
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int f = blockIdx.y * 4 + warp; f < a.F; f += gridDim.y * 4) {
    const E *pg = wg + ((size_t)g * a.F + f) * a.H;
    const E *pu = wu + ((size_t)g * a.F + f) * a.H;
    float ag = 0.f, au = 0.f;
    for (int k = lane; k < a.H; k += 32) {
      ag = fmaf(to_f<E>(pg[k]), hs[k], ag);
      au = fmaf(to_f<E>(pu[k]), hs[k], au);
    }
    ag = warp_sum(ag);
    au = warp_sum(au);
    if (lane == 0) U[(size_t)row * a.F + f] = from_f<E>(ag / (1.0f + expf(-ag)) * au);
  }
}

template <typename E>
__global__ void __launch_bounds__(128) simt_stage2_kernel(const SimtArgs a, const E *U, const E *wd,
                                                          float *y) {
  extern __shared__ float as[];
  __shared__ int sg, srow, stok;
  __shared__ float sw;
  const int row = blockIdx.x;
  if (threadIdx.x == 0) {
    sg = a.offsets ? find_group(a.offsets, a.G, row) : (row < a.rows ? 0 : -1);
    int ur = sg < 0 ? 0 : (a.row_src ? a.row_src[row] : row);
    int tok = sg < 0 ? 0 : (a.row_token ? a.row_token[row] : row);
    if ((unsigned)ur >= (unsigned)a.limit_src || (unsigned)tok >= (unsigned)a.T) {
      atomicCAS(&a.plan->status, 0, PCOMOE_ERR_INDEX);
      sg = -1;
    }
    srow = ur;
    stok = tok;
    sw = (sg >= 0 && a.row_w) ? a.row_w[row] : 1.0f;
  }
  __syncthreads();
  const int g = sg;
  if (g < 0) return;
  const E *ur = U + (size_t)srow * a.F;
  for (int k = threadIdx.x; k < a.F; k += blockDim.x) as[k] = to_f<E>(ur[k]);
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int c = blockIdx.y * 4 + warp; c < a.H; c += gridDim.y * 4) {
    const E *pw = wd + ((size_t)g * a.H + c) * a.F;
    float acc = 0.f;
    for (int k = lane; k < a.F; k += 32) acc = fmaf(to_f<E>(pw[k]), as[k], acc);
    acc = warp_sum(acc);
    if (lane == 0) atomicAdd(&y[(size_t)stok * a.H + c], sw * acc);
  }
}

template <typename E>
static pcomoe_status run_simt(const pcomoe_layer *L, int32_t T, const void *h, const void *wg,
                              const void *wu, const void *wd, const void *sg, const void *su,
                              const void *sd, const pcomoe_groups *g, float *y, char *ws,
                              const WsLayout &lay, cudaStream_t st, int stages) {
  const pcomoe_config &c = L->cfg;
  DevPlan *plan = reinterpret_cast<DevPlan *>(ws + lay.plan);
  E *U = reinterpret_cast<E *>(ws + lay.u);
  E *Ush = reinterpret_cast<E *>(ws + lay.u_sh);
  const int P = T * c.top_k;
  SimtArgs a1{};
  a1.offsets = g->s1_offsets; a1.row_src = g->s1_token; a1.G = c.n_experts; a1.rows = P;
  a1.H = c.hidden; a1.F = c.ffn; a1.limit_src = T; a1.T = T; a1.plan = plan;
  const int gy1 = max(1, min(16, c.ffn / 64));
  if (stages & kStage1Routed) {
    simt_stage1_kernel<E><<<dim3(P, gy1), 128, sizeof(float) * c.hidden, st>>>(
        a1, (const E *)h, (const E *)wg, (const E *)wu, U);
    count_launch();
  }

  SimtArgs a2{};
  a2.offsets = g->s2_offsets; a2.row_src = g->s2_s1row; a2.row_token = g->s2_token; a2.row_w = g->s2_w;
  a2.G = c.n_experts; a2.rows = P; a2.H = c.hidden; a2.F = c.ffn; a2.limit_src = P; a2.T = T; a2.plan = plan;
  const int gy2 = max(1, min(16, c.hidden / 64));
  if (stages & kStage2Routed) {
    PCOMOE_CUDA_TRY(cudaMemsetAsync(y, 0, sizeof(float) * (size_t)T * c.hidden, st));
    simt_stage2_kernel<E><<<dim3(P, gy2), 128, sizeof(float) * c.ffn, st>>>(a2, U, (const E *)wd, y);
    count_launch(2);
  }

  if (c.shared_ffn > 0) {
    SimtArgs s1{};
    s1.G = 1; s1.rows = T; s1.H = c.hidden; s1.F = c.shared_ffn; s1.limit_src = T; s1.T = T; s1.plan = plan;
    const int gy = max(1, min(16, c.shared_ffn / 64));
    if (stages & kStage1Shared) {
      simt_stage1_kernel<E><<<dim3(T, gy), 128, sizeof(float) * c.hidden, st>>>(
          s1, (const E *)h, (const E *)sg, (const E *)su, Ush);
      count_launch();
    }
    SimtArgs s2 = s1;
    if (stages & kStage2Shared) {
      simt_stage2_kernel<E><<<dim3(T, gy2), 128, sizeof(float) * c.shared_ffn, st>>>(s2, Ush, (const E *)sd, y);
      count_launch();
    }
  }
  PCOMOE_CUDA_TRY(cudaGetLastError());
  return PCOMOE_OK;
}

pcomoe_status launch_ffn_simt(const pcomoe_layer *L, int32_t T, const void *h, const void *wg,
                              const void *wu, const void *wd, const void *sg, const void *su,
                              const void *sd, const pcomoe_groups *g, float *y, char *ws,
                              const WsLayout &lay, cudaStream_t st, int stages) {
  const size_t need = sizeof(float) * (size_t)max(max(L->cfg.hidden, L->cfg.ffn), L->cfg.shared_ffn);
  if (need > 200 * 1024) return PCOMOE_ERR_UNSUPPORTED;
  if (need > 48 * 1024) {
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(simt_stage1_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need));
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(simt_stage2_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need));
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(simt_stage1_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need));
    PCOMOE_CUDA_TRY(cudaFuncSetAttribute(simt_stage2_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need));
  }
  if (L->cfg.in_dtype == PCOMOE_FP32)
    return run_simt<float>(L, T, h, wg, wu, wd, sg, su, sd, g, y, ws, lay, st, stages);
  return run_simt<__nv_bfloat16>(L, T, h, wg, wu, wd, sg, su, sd, g, y, ws, lay, st, stages);
}

}  // namespace pcomoe
