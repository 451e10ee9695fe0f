// Internal declarations shared by the translation units of libpcomoe.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "pcomoe.h"

namespace pcomoe {

constexpr int kTileM = 128;        // rows of one GEMM tile (one TMEM lane per row)
constexpr int kMaxExperts = 256;
constexpr int kMaxTopK = 32;

// One entry of the active-path table (sorted by flat id src*n+tgt).
struct __align__(8) ActiveEntry {
  uint16_t src;
  uint16_t tgt;
  float bias;
};

// Device-side header at the start of the workspace.
struct DevPlan {
  int32_t status;      // first device-detected error (pcomoe_status), 0 if none
  int32_t R1;          // stage-1 rows
  int32_t P;           // stage-2 rows (= T*K)
  int32_t mt1;         // 128-row tiles of stage 1 (sum over sources of ceil(rows/128))
  int32_t mt2;         // 128-row tiles of stage 2
  int32_t empty1;      // sources without rows
  int32_t empty2;      // targets without rows
  int32_t T;           // tokens of the last pcomoe_build_path_groups
  int32_t status_router;   // first error of the router kernel; not cleared by the grouping step
};
constexpr size_t kPlanClearBytes = 32;   // what the grouping step zeroes: everything before status_router

// Byte offsets of the workspace sections (all multiples of 256).
struct WsLayout {
  size_t plan;         // DevPlan
  size_t tile_base1;   // int32 [n+1]   prefix of stage-1 m-tiles per source
  size_t tile_base2;   // int32 [n+1]   prefix of stage-2 m-tiles per target
  size_t col_tot;      // int32 [2][n]     rows per (stage, expert)
  size_t blk_cnt;      // int32 [2][n][NB] per-block histograms, turned into offsets by the scan
  size_t a1_idx;       // int32 [mt_max*128] token of every padded stage-1 row (0 in the padding)
  size_t path_prow1;   // int32 [T*K] padded stage-1 row of every path
  size_t path_pos2;    // int32 [T*K] padded stage-2 row of every path
  size_t u;            // in_dtype [mt_max*128, F]   intermediates (tensor-core path: in padded stage-2
                       //                            order; SIMT path: by unpadded stage-1 row)
  size_t u_sh;         // in_dtype [Tpad, F_sh]      shared-expert intermediates
  size_t h_gath;       // bf16 [mt_max*128, H]       rows of h in padded stage-1 order (tensor-core path)
  size_t path_wgt;     // fp32 [T*K]                 copy of the path weights (projection-side reuse only)
  size_t y_acc;        // fp32 [T, H]                fp32 accumulator of y when the layer's output type is bf16
  size_t total;
  int32_t nb_max;      // blocks of the grouping kernels at max_tokens
  int32_t mt_max;      // upper bound of m-tiles per stage
  int32_t t_pad;       // max_tokens rounded up to 128
};

}  // namespace pcomoe

struct pcomoe_layer {
  pcomoe_config cfg;
  int32_t n_active;                 // |A|
  pcomoe::ActiveEntry *d_table;     // device copy of the active-path table
  pcomoe::ActiveEntry *h_table;     // host copy
  int device;
  int sm_count;
  int group_chunk;                  // tokens per block of the grouping kernels
  int tc_ok;                        // sizes and dtype allow the tcgen05 path
  cudaStream_t side_stream;         // pcomoe_layer_forward: the shared expert's stage 1 runs here beside the routing chain
  cudaEvent_t ev_fork, ev_join;     //                       ordering of side_stream against the caller's stream
};

namespace pcomoe {

WsLayout ws_layout(const pcomoe_layer *L, int32_t max_tokens);
void count_launch(int n = 1);
uint64_t wait_limit_ns();            // limit of every bounded device-side wait (pcomoe_set_wait_limit_us)

inline size_t dtype_size(int dt) { return dt == PCOMOE_BF16 ? 2 : 4; }

// Tokens per block of the grouping kernels for a batch of T tokens: the largest chunk the layer allows
// (shared-memory bound), halved while that would leave fewer than two blocks per SM.
// CTA pairs pay off once groups are a few tiles long; short groups (decode) leave the peer CTA idle
inline bool use_cta_pairs(const pcomoe_layer *L, int32_t T) {
  const pcomoe_config &c = L->cfg;
  return c.ffn_impl == PCOMOE_FFN_TCGEN05_PAIR ||
         (c.ffn_impl == PCOMOE_FFN_AUTO && (int64_t)T * c.top_k >= (int64_t)256 * c.n_experts);
}

inline int group_chunk_for(const pcomoe_layer *L, int32_t T) {
  int chunk = L->group_chunk;
  if (T <= chunk) return chunk;   // the whole batch fits one block
  while (chunk > 32 && (int64_t)T / chunk < 2 * (int64_t)L->sm_count) chunk >>= 1;
  return chunk;
}

// Kernel attributes (cudaFuncSetAttribute) belong to a device: a once-flag per device ordinal.  first_use()
// is true until done() has been called for that device; setting the attributes twice is harmless, so a race
// between two threads only repeats the calls.  Devices beyond the table set their attributes on every call.
struct PerDeviceOnce {
  std::atomic<uint64_t> mask{0};
  bool first_use(int device) const {
    return device < 0 || device >= 64 || !((mask.load(std::memory_order_acquire) >> device) & 1u);
  }
  void done(int device) {
    if (device >= 0 && device < 64) mask.fetch_or(uint64_t(1) << device, std::memory_order_release);
  }
};

#define PCOMOE_CUDA_TRY(expr)                          \
  do {                                                 \
    cudaError_t _e = (expr);                           \
    if (_e != cudaSuccess) return PCOMOE_ERR_CUDA;     \
  } while (0)

// Programmatic dependent launch.  Every kernel of the library begins with pdl_grid_wait(), which holds it until
// the kernel before it in the stream has completed and its writes are visible, and then lets the kernel after it
// start its own launch and prologue early (it will block in its own pdl_grid_wait()).  Launched with
// launch_pdl(), consecutive kernels of a call overlap their launch latencies instead of adding them.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_grid_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// launchers implemented in the kernel translation units
pcomoe_status launch_route(const pcomoe_layer *L, int32_t T, const float *z, const float *u,
                           int32_t *src, int32_t *tgt, float *w, cudaStream_t st);
pcomoe_status launch_router(const pcomoe_layer *L, int32_t T, const void *h, const void *w_router,
                            const void *lora_a, const float *lora_b, int32_t r, float scale, float *logits,
                            int32_t *status, cudaStream_t st);
pcomoe_status launch_cast_y(const pcomoe_layer *L, int32_t T, const float *y_acc, void *y_out, cudaStream_t st);
pcomoe_status launch_wait_probe(int32_t *status_word, cudaStream_t st);
pcomoe_status launch_residual_cast(const pcomoe_layer *L, int32_t T, const void *h_in, const float *y, void *h_out,
                                   cudaStream_t st);
pcomoe_status launch_groups(const pcomoe_layer *L, int32_t T, const int32_t *src, const int32_t *tgt,
                            const float *w, const pcomoe_groups *g, char *ws, const WsLayout &lay,
                            cudaStream_t st);
pcomoe_status launch_ffn_simt(const pcomoe_layer *L, int32_t T, const void *h, const void *wg,
                              const void *wu, const void *wd, const void *sg, const void *su,
                              const void *sd, const pcomoe_groups *g, float *y, char *ws,
                              const WsLayout &lay, cudaStream_t st, int stages);
pcomoe_status launch_shared_stage1_side(const pcomoe_layer *L, int32_t T, const void *h, const void *sg,
                                        const void *su, char *ws, const WsLayout &lay, cudaStream_t st, int32_t rows);
pcomoe_status launch_ffn_tc(const pcomoe_layer *L, int32_t T, const void *h, const void *wg,
                            const void *wu, const void *wd, const void *sg, const void *su,
                            const void *sd, const pcomoe_groups *g, float *y, char *ws,
                            const WsLayout &lay, cudaStream_t st, int stages,
                            cudaEvent_t wait_before_stage2 = nullptr, int32_t shared_row0 = 0);

// bits of `stages`
constexpr int kStage1Routed = 1, kStage1Shared = 2, kStage2Routed = 4, kStage2Shared = 8;

}  // namespace pcomoe
