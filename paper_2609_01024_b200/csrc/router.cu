// K0: the router in front of the path gate (Sec. 3.1: the router turns a token's hidden state into routing
// scores; Sec. 4.2 calls them the base routing signal g_base(h)):
//     logits[t,e] = sum_k h[t,k] W_r[e,k]   (+ scale * sum_q B_l[e,q] * sum_k A_l[q,k] h[t,k], the rank-r gate
//                                              adaptation of Sec. 5.1)
// The work is a skinny GEMM bound by one read of h, so a tile is 128 tokens x all experts: a CTA streams rows of
// h through a deep TMA ring (a stage is 16 KB of h plus the few weight rows, so up to 12 stages are in flight)
// while W_r (and A_l, stacked under it as extra output columns) comes from L2, one thread issues tcgen05.mma
// (M 128, N = padded n + r, bf16 in, fp32 accumulate in TMEM), and the epilogue turns the accumulators around
// through shared memory, applies the low-rank term and writes fp32 logits coalesced.  When the batch has few
// tiles, a cluster of 2, 4 or 8 CTAs shares each tile along K and adds the partial sums through distributed
// shared memory in rank order: no atomics, so for a given batch size the logits are reproducible bit for bit,
// which matters because they decide the TopK.
// Layers that are not bf16 (or whose shapes the tile does not cover) take a plain SIMT kernel.
#include <cuda_bf16.h>

#include "tc_ptx.cuh"

namespace pcomoe {
namespace {

constexpr int kRMaxStages = 12;
constexpr uint32_t kRA = kTileM * BK * 2;            // 16 KB of h per k-block
constexpr size_t kRSmem = 196 * 1024 + 1024;         // ring (and, after the MMAs, the turn-around buffers)
constexpr int kRThreads = 192;

struct RouterParams {
  float *logits;          // [T,n]
  const float *lora_b;    // [n,r] or NULL
  int32_t *status;        // device status word of the router (may be NULL)
  int32_t T, n, r, n8;    // n8: row of the stacked tile where A_l starts (n rounded up to 8)
  int32_t n_mma;          // MMA N: n8 + r rounded up to 16
  int32_t kb;             // k-blocks
  int32_t split;          // CTAs of a cluster that share one tile, each taking a slice of the k-blocks
  int32_t stages;         // ring depth
  uint32_t stage_bytes;   // kRA + n_mma * 128
  uint32_t idesc, tmem_cols;
  float scale;
  uint64_t wait_ns;       // limit of every mbarrier wait
};

__device__ __forceinline__ void umma_bf16_n(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ uint32_t rank_in_cluster() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// fp32 word at shared-memory address `local_addr` of the cluster's CTA `rank`
__device__ __forceinline__ float ld_peer_f32(uint32_t local_addr, uint32_t rank) {
  uint32_t ra;
  float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
  return v;
}

// A cluster of `split` CTAs owns one tile of 128 tokens; CTA c of the cluster multiplies k-blocks
// [c*kb/split, (c+1)*kb/split) and the partial accumulators are added through distributed shared memory in
// rank order, so the sum does not depend on timing.
__global__ void __launch_bounds__(kRThreads, 1)
router_gemm_kernel(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmW,
                   const __grid_constant__ CUtensorMap tmL, const RouterParams p) {
  extern __shared__ unsigned char smem_dyn[];
  pdl_grid_wait();
  __shared__ __align__(8) uint64_t s_bar[2 * kRMaxStages + 1];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ float s_lb[64 * 64];                      // B_l transposed to [r][n] when it fits (n*r <= 4096), else global

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t ring = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char *ring_ptr = smem_dyn + (ring - smem_u32(smem_dyn));
  const uint32_t bar0 = smem_u32(s_bar);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kRMaxStages + s); };
  const uint32_t acc_bar = bar0 + 8u * (2 * kRMaxStages);
  const bool lb_smem = p.r > 0 && p.n * p.r <= 64 * 64;
  const int crank = p.split > 1 ? (int)rank_in_cluster() : 0;
  const int tile = blockIdx.x / p.split;
  const int kb_lo = (int)((int64_t)crank * p.kb / p.split), kb_hi = (int)((int64_t)(crank + 1) * p.kb / p.split);

  // rows of the stacked weight tile that no load writes (padding up to the MMA's N) start as zeros
  for (int s = 0; s < p.stages; ++s) {
    uint4 *b = reinterpret_cast<uint4 *>(ring_ptr + (size_t)s * p.stage_bytes + kRA);
    for (int i = threadIdx.x; i < p.n_mma * 8; i += blockDim.x) b[i] = make_uint4(0, 0, 0, 0);
  }
  if (lb_smem)
    for (int i = threadIdx.x; i < p.n * p.r; i += blockDim.x) s_lb[(i % p.r) * p.n + i / p.r] = p.lora_b[i];
  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(acc_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem;
  volatile int *abort_flag = &s_abort;
  const int row0 = tile * kTileM;
  const uint32_t stage_tx = kRA + (uint32_t)(p.n + p.r) * (BK * 2);

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int kb = kb_lo; kb < kb_hi; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.wait_ns)) break;
        const uint32_t sa = ring + stage * p.stage_bytes, sb = sa + kRA;
        mbar_arrive_expect_tx(full_bar(stage), stage_tx);
        tma_load_2d(sa, &tmH, kb * BK, row0, full_bar(stage));
        tma_load_2d(sb, &tmW, kb * BK, 0, full_bar(stage));
        if (p.r > 0) tma_load_2d(sb + (uint32_t)p.n8 * (BK * 2), &tmL, kb * BK, 0, full_bar(stage));
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool alive = true;
      for (int kb = kb_lo; kb < kb_hi; ++kb) {
        if (!mbar_wait(full_bar(stage), phase, abort_flag, p.wait_ns)) { alive = false; break; }
        tc_fence_after();
        const uint32_t sa = ring + stage * p.stage_bytes, sb = sa + kRA;
        const uint64_t da = umma_desc(sa), db = umma_desc(sb);
#pragma unroll
        for (int k = 0; k < BK / 16; ++k)
          umma_bf16_n(tmem_base, da + 2u * k, db + 2u * k, p.idesc, (kb > kb_lo || k != 0) ? 1u : 0u);
        umma_commit(empty_bar(stage));
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
      }
      if (alive) umma_commit(acc_bar);
    }
    __syncwarp();
  }
  // every thread waits for the accumulator: the ring is free after that and becomes the turn-around buffer
  const bool done = mbar_wait(acc_bar, 0, abort_flag, p.wait_ns);
  tc_fence_after();
  __syncthreads();
  float *turn = reinterpret_cast<float *>(ring_ptr);          // [128][n_mma + 1] fp32: this CTA's partial sums
  const int ld = p.n_mma + 1;
  if (done && !s_abort) {
    if (warp >= 2) {
      const int quarter = warp & 3;
      const int r = quarter * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
      uint32_t v[32];
      for (int c0 = 0; c0 < p.n_mma; c0 += 32) {
        tmem_ld32_issue(taddr + c0, v);
        tmem_wait_ld();
        reg_fence32(v);
#pragma unroll
        for (int c = 0; c < 32; ++c)
          if (c0 + c < p.n_mma) turn[r * ld + c0 + c] = __uint_as_float(v[c]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  // rows of the tile this CTA finishes: an equal share per CTA of the cluster
  const int share = kTileM / p.split;
  const int r_lo = crank * share;
  const float *sums = turn;                                   // [.][ld], indexed by tile row
  if (p.split > 1) {
    cluster_barrier();                                        // every CTA's partial sums are in place
    float *red = turn + kTileM * ld;                          // [share][ld]: the cluster's sums for this CTA's rows
    const uint32_t turn_addr = ring;
    for (int i = threadIdx.x; i < share * p.n_mma; i += blockDim.x) {
      const int rr = i / p.n_mma, c = i - rr * p.n_mma;
      const uint32_t off = (uint32_t)(((r_lo + rr) * ld + c) * 4);
      float acc = 0.0f;
      for (int s = 0; s < p.split; ++s) acc += ld_peer_f32(turn_addr + off, (uint32_t)s);
      red[rr * ld + c] = acc;
    }
    __syncthreads();
    sums = red - r_lo * ld;                                   // so that sums[r * ld + c] addresses tile row r
  }
  if (done && !s_abort) {
    const int rows = min(kTileM, p.T - row0);
    const int r_hi = min(rows, r_lo + share);
    const int total = (r_hi - r_lo) * p.n;
    float *out = p.logits + ((size_t)row0 + r_lo) * p.n;
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
      const int r = r_lo + i / p.n, e = i % p.n;
      float v = sums[r * ld + e];
      if (p.r > 0) {
        const float *low = sums + r * ld + p.n8;
        float d = 0.0f;
        if (lb_smem) {   // neighbouring threads hold neighbouring experts: [r][n] keeps their reads on separate banks
          for (int q = 0; q < p.r; ++q) d = fmaf(s_lb[q * p.n + e], low[q], d);
        } else {
          const float *bl = p.lora_b + (size_t)e * p.r;
          for (int q = 0; q < p.r; ++q) d = fmaf(bl[q], low[q], d);
        }
        v = fmaf(p.scale, d, v);
      }
      out[i] = v;
    }
  }
  if (p.split > 1) cluster_barrier();                         // peers may still be reading this CTA's sums
  // ---------------- teardown ----------------
  if (s_abort) {
    if (p.status) timeout_record_and_drain(p.status);
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}

// Plain kernel for fp32 layers and shapes the tile does not cover: one block per token; the hidden row is staged
// in shared memory as fp32, warps take the low-rank rows and then the experts in turn, lanes stride over H.
template <typename TIn>
__device__ __forceinline__ float to_f32(TIn v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename TIn>
__global__ void __launch_bounds__(128) router_simt_kernel(const TIn *h, const TIn *w, const TIn *la, const float *lb,
                                                          float *logits, int T, int H, int n, int r, float scale) {
  extern __shared__ float s_row[];      // [H] hidden row, then [r] low-rank activations
  pdl_grid_wait();
  float *low = s_row + H;
  const int t = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
  for (int k = threadIdx.x; k < H; k += blockDim.x) s_row[k] = to_f32<TIn>(h[(size_t)t * H + k]);
  __syncthreads();
  for (int q = warp; q < r; q += warps) {
    float acc = 0.0f;
    for (int k = lane; k < H; k += 32) acc = fmaf(to_f32<TIn>(la[(size_t)q * H + k]), s_row[k], acc);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) low[q] = acc;
  }
  __syncthreads();
  for (int e = warp; e < n; e += warps) {
    float acc = 0.0f;
    for (int k = lane; k < H; k += 32) acc = fmaf(to_f32<TIn>(w[(size_t)e * H + k]), s_row[k], acc);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) {
      float d = 0.0f;
      for (int q = 0; q < r; ++q) d = fmaf(lb[(size_t)e * r + q], low[q], d);
      logits[(size_t)t * n + e] = fmaf(scale, d, acc);
    }
  }
}

}  // namespace

pcomoe_status launch_router(const pcomoe_layer *L, int32_t T, const void *h, const void *w_router,
                            const void *lora_a, const float *lora_b, int32_t r, float scale, float *logits,
                            int32_t *status, cudaStream_t st) {
  const pcomoe_config &c = L->cfg;
  const int n = c.n_experts, H = c.hidden;
  const int n8 = (n + 7) & ~7;
  const int n_mma = (n8 + r + 15) & ~15;
  const bool tc = c.in_dtype == PCOMOE_BF16 && c.ffn_impl != PCOMOE_FFN_SIMT && H % 8 == 0 && H >= BK &&
                  n_mma <= 256 && r <= 64;
  if (tc) {
    CUtensorMap mH, mW, mL;
    bool ok = make_map(&mH, h, (uint64_t)T, H, kTileM) && make_map(&mW, w_router, (uint64_t)n, H, (uint32_t)n);
    if (ok && r > 0) ok = make_map(&mL, lora_a, (uint64_t)r, H, (uint32_t)r);
    if (!ok) return PCOMOE_ERR_CUDA;
    if (r == 0) mL = mW;
    RouterParams p{};
    p.logits = logits; p.lora_b = lora_b; p.status = status;
    p.T = T; p.n = n; p.r = r; p.n8 = n8; p.n_mma = n_mma; p.kb = (H + BK - 1) / BK;
    p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)n_mma >> 3) << 17) | ((128u >> 4) << 24);
    p.tmem_cols = n_mma <= 32 ? 32u : n_mma <= 64 ? 64u : n_mma <= 128 ? 128u : 256u;
    p.scale = scale;
    p.wait_ns = wait_limit_ns();
    p.stage_bytes = kRA + (uint32_t)n_mma * (BK * 2);
    p.stages = (int)((kRSmem - 1024) / p.stage_bytes);
    if (p.stages > kRMaxStages) p.stages = kRMaxStages;
    // few tiles: a cluster shares each tile along K so that more SMs stream h (powers of two up to 8, at least
    // two k-blocks per CTA, and only while the partial sums of a cluster fit next to the reduced rows)
    const int tiles = (T + kTileM - 1) / kTileM;
    int split = 1;
    while (split < 8 && tiles * split * 2 <= L->sm_count && p.kb >= 4 * split && n_mma <= 128) split *= 2;
    p.split = split;
    static PerDeviceOnce attr_once;
    if (attr_once.first_use(L->device)) {
      PCOMOE_CUDA_TRY(cudaFuncSetAttribute(router_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRSmem));
      attr_once.done(L->device);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(tiles * split);
    cfg.blockDim = dim3(kRThreads);
    cfg.dynamicSmemBytes = kRSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = split;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = split > 1 ? 2 : 1;
    PCOMOE_CUDA_TRY(cudaLaunchKernelEx(&cfg, router_gemm_kernel, mH, mW, mL, p));
  } else {
    const size_t smem = sizeof(float) * ((size_t)H + (r > 0 ? r : 1));
    if (smem > 200 * 1024) return PCOMOE_ERR_UNSUPPORTED;
    if (c.in_dtype == PCOMOE_BF16) {
      auto k = router_simt_kernel<__nv_bfloat16>;
      if (smem > 48 * 1024) PCOMOE_CUDA_TRY(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      PCOMOE_CUDA_TRY(launch_pdl(k, dim3(T), dim3(128), smem, st, (const __nv_bfloat16 *)h, (const __nv_bfloat16 *)w_router,
                                 (const __nv_bfloat16 *)lora_a, lora_b, logits, (int)T, H, n, (int)r, scale));
    } else {
      auto k = router_simt_kernel<float>;
      if (smem > 48 * 1024) PCOMOE_CUDA_TRY(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      PCOMOE_CUDA_TRY(launch_pdl(k, dim3(T), dim3(128), smem, st, (const float *)h, (const float *)w_router,
                                 (const float *)lora_a, lora_b, logits, (int)T, H, n, (int)r, scale));
    }
  }
  count_launch();
  PCOMOE_CUDA_TRY(cudaGetLastError());
  return PCOMOE_OK;
}

}  // namespace pcomoe
