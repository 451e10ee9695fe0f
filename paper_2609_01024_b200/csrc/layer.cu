// Host side of the C ABI: layer set-up, workspace sizing, argument checks and dispatch.
#include <cstddef>
#include <algorithm>
#include <atomic>
#include <cmath>
#include <vector>
#include <cstdlib>
#include <cstring>
#include <new>

#include "common.cuh"

using namespace pcomoe;

namespace pcomoe {

static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static std::atomic<uint64_t> g_wait_limit_ns{2000000000ull};   // 2 s
uint64_t wait_limit_ns() { return g_wait_limit_ns.load(std::memory_order_relaxed); }

static size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

WsLayout ws_layout(const pcomoe_layer *L, int32_t max_tokens) {
  const pcomoe_config &c = L->cfg;
  WsLayout w{};
  const int64_t Tm = max_tokens > 0 ? max_tokens : 1;
  const int64_t Pm = Tm * c.top_k;
  // upper bound of the grouping kernels' block count for any batch up to Tm (see group_chunk_for)
  const int64_t nb_small = (Tm + 31) / 32 < 4 * (int64_t)L->sm_count ? (Tm + 31) / 32 : 4 * (int64_t)L->sm_count;
  const int64_t nb_large = (Tm + L->group_chunk - 1) / L->group_chunk;
  w.nb_max = (int32_t)(nb_small > nb_large ? nb_small : nb_large);
  w.mt_max = (int32_t)(Pm / kTileM + c.n_experts + 1);
  w.t_pad = (int32_t)((Tm + kTileM - 1) / kTileM * kTileM);
  const size_t es = dtype_size(c.in_dtype);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align256(off + bytes);
    return o;
  };
  w.plan = take(sizeof(DevPlan));
  w.tile_base1 = take(sizeof(int32_t) * (c.n_experts + 1));
  w.tile_base2 = take(sizeof(int32_t) * (c.n_experts + 1));
  w.col_tot = take(sizeof(int32_t) * 2 * c.n_experts);
  w.blk_cnt = take(sizeof(int32_t) * (size_t)w.nb_max * 2 * c.n_experts);
  w.a1_idx = take(sizeof(int32_t) * (size_t)w.mt_max * kTileM);
  w.path_prow1 = take(sizeof(int32_t) * (size_t)Pm);
  w.path_pos2 = take(sizeof(int32_t) * (size_t)Pm);
  w.u = take(es * (size_t)w.mt_max * kTileM * c.ffn);
  w.u_sh = take(es * (size_t)w.t_pad * c.shared_ffn);
  if (L->tc_ok) w.h_gath = take(es * (size_t)w.mt_max * kTileM * c.hidden);
  if (c.target_reuse) w.path_wgt = take(sizeof(float) * (size_t)Pm);
  if (c.out_dtype == PCOMOE_BF16) w.y_acc = take(sizeof(float) * (size_t)Tm * c.hidden);
  w.total = off;
  return w;
}

}  // namespace pcomoe

extern "C" {

pcomoe_status pcomoe_layer_create(const pcomoe_config *cfg, const uint8_t *h_mask,
                                  const float *h_bias, pcomoe_layer **out) {
  if (!cfg || !h_mask || !h_bias || !out) return PCOMOE_ERR_INVALID_ARG;
  // the struct may end before `target_reuse` (the layout before that field was added)
  const int32_t old_size = (int32_t)offsetof(pcomoe_config, target_reuse);
  if (cfg->struct_size != (int32_t)sizeof(pcomoe_config) && cfg->struct_size != old_size) return PCOMOE_ERR_INVALID_ARG;
  pcomoe_config full = {};
  std::memcpy(&full, cfg, (size_t)cfg->struct_size);
  full.struct_size = (int32_t)sizeof(pcomoe_config);
  cfg = &full;
  if (cfg->target_reuse != 0 && cfg->target_reuse != 1) return PCOMOE_ERR_INVALID_ARG;
  const int n = cfg->n_experts, K = cfg->top_k;
  if (n <= 0 || K <= 0 || cfg->hidden <= 0 || cfg->ffn <= 0 || cfg->shared_ffn < 0)
    return PCOMOE_ERR_INVALID_ARG;
  if (cfg->in_dtype != PCOMOE_BF16 && cfg->in_dtype != PCOMOE_FP32) return PCOMOE_ERR_INVALID_ARG;
  if (cfg->ffn_impl < PCOMOE_FFN_AUTO || cfg->ffn_impl > PCOMOE_FFN_TCGEN05_PAIR)
    return PCOMOE_ERR_INVALID_ARG;
  if (K > n || K > kMaxTopK) return PCOMOE_ERR_SHAPE;
  if (n > kMaxExperts) return PCOMOE_ERR_UNSUPPORTED;
  if (cfg->out_dtype != PCOMOE_FP32 && cfg->out_dtype != PCOMOE_BF16) return PCOMOE_ERR_INVALID_ARG;
  if (cfg->hidden % 8 || cfg->ffn % 8 || cfg->shared_ffn % 8) return PCOMOE_ERR_UNSUPPORTED;
  for (int i = 0; i < n; ++i)
    if (!h_mask[(size_t)i * n + i]) return PCOMOE_ERR_INVALID_ARG;  // m_ii = 1 (Sec. 4.2)

  pcomoe_layer *L = new (std::nothrow) pcomoe_layer();
  if (!L) return PCOMOE_ERR_CUDA;
  L->cfg = *cfg;
  L->tc_ok = cfg->in_dtype == PCOMOE_BF16 && cfg->hidden % 256 == 0 && cfg->ffn % 128 == 0 &&
             cfg->shared_ffn % 128 == 0;
  if (cfg->ffn_impl >= PCOMOE_FFN_TCGEN05 && !L->tc_ok) {
    delete L;
    return PCOMOE_ERR_UNSUPPORTED;
  }
  // projection-side reuse lives in the tensor-core epilogue only
  if (cfg->target_reuse && (!L->tc_ok || cfg->ffn_impl == PCOMOE_FFN_SIMT)) {
    delete L;
    return PCOMOE_ERR_UNSUPPORTED;
  }

  int cnt = 0;
  for (int i = 0; i < n * n; ++i) cnt += h_mask[i] ? 1 : 0;
  L->n_active = cnt;
  L->h_table = (ActiveEntry *)std::malloc(sizeof(ActiveEntry) * (size_t)cnt);
  if (!L->h_table) {
    delete L;
    return PCOMOE_ERR_CUDA;
  }
  int a = 0;
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < n; ++j)
      if (h_mask[(size_t)i * n + j]) {
        L->h_table[a].src = (uint16_t)i;
        L->h_table[a].tgt = (uint16_t)j;
        L->h_table[a].bias = h_bias[(size_t)i * n + j];
        ++a;
      }

  // tokens per block of the grouping kernels: the two bit matrices [n][chunk*K/32] must fit
  int chunk = 128;
  auto scatter_smem = [&](int ch) {
    const size_t ck = (size_t)ch * K, words = (ck + 31) / 32;
    return 4 * (4 * ck + 6 * (size_t)n + 2 * (size_t)n * words);
  };
  while (chunk > 32 && scatter_smem(chunk) > 96 * 1024) chunk >>= 1;
  L->group_chunk = chunk;

  cudaError_t e = cudaGetDevice(&L->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&L->sm_count, cudaDevAttrMultiProcessorCount, L->device);
  if (e == cudaSuccess) e = cudaMalloc((void **)&L->d_table, sizeof(ActiveEntry) * (size_t)cnt);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&L->side_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&L->ev_fork, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&L->ev_join, cudaEventDisableTiming);
  if (e == cudaSuccess)
    e = cudaMemcpy(L->d_table, L->h_table, sizeof(ActiveEntry) * (size_t)cnt, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    if (L->d_table) cudaFree(L->d_table);
    if (L->side_stream) cudaStreamDestroy(L->side_stream);
    if (L->ev_fork) cudaEventDestroy(L->ev_fork);
    if (L->ev_join) cudaEventDestroy(L->ev_join);
    std::free(L->h_table);
    delete L;
    return PCOMOE_ERR_CUDA;
  }
  *out = L;
  return PCOMOE_OK;
}

pcomoe_status pcomoe_mask_from_bias(int32_t n, const float *h_bias, float keep_fraction, uint8_t *h_mask) {
  if (n <= 0 || !h_bias || !h_mask || !(keep_fraction >= 0.0f && keep_fraction <= 1.0f)) return PCOMOE_ERR_INVALID_ARG;
  const int64_t off = (int64_t)n * (n - 1);
  const int64_t keep = (int64_t)std::llround((double)keep_fraction * (double)off);
  std::vector<int32_t> order;
  order.reserve((size_t)off);
  for (int32_t i = 0; i < n; ++i)
    for (int32_t j = 0; j < n; ++j)
      if (i != j) order.push_back(i * n + j);
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return h_bias[a] > h_bias[b]; });
  std::memset(h_mask, 0, (size_t)n * n);
  for (int32_t i = 0; i < n; ++i) h_mask[(size_t)i * n + i] = 1;
  for (int64_t r = 0; r < keep; ++r) h_mask[order[(size_t)r]] = 1;
  return PCOMOE_OK;
}

pcomoe_status pcomoe_mask_tighten(int32_t n, const float *h_bias, const uint8_t *h_prev_mask, float keep_fraction,
                                  uint8_t *h_mask) {
  if (n <= 0 || !h_bias || !h_prev_mask || !h_mask || !(keep_fraction >= 0.0f && keep_fraction <= 1.0f))
    return PCOMOE_ERR_INVALID_ARG;
  std::vector<int32_t> order;
  for (int32_t i = 0; i < n; ++i)
    for (int32_t j = 0; j < n; ++j)
      if (i != j && h_prev_mask[(size_t)i * n + j]) order.push_back(i * n + j);
  const int64_t keep = (int64_t)std::llround((double)keep_fraction * (double)order.size());
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return h_bias[a] > h_bias[b]; });
  std::vector<uint8_t> m((size_t)n * n, 0);          // built aside: h_mask may be h_prev_mask
  for (int32_t i = 0; i < n; ++i) m[(size_t)i * n + i] = 1;
  for (int64_t r = 0; r < keep; ++r) m[(size_t)order[(size_t)r]] = 1;
  std::memcpy(h_mask, m.data(), m.size());
  return PCOMOE_OK;
}

pcomoe_status pcomoe_layer_destroy(pcomoe_layer *L) {
  if (!L) return PCOMOE_ERR_INVALID_ARG;
  if (L->d_table) cudaFree(L->d_table);
  if (L->side_stream) cudaStreamDestroy(L->side_stream);
  if (L->ev_fork) cudaEventDestroy(L->ev_fork);
  if (L->ev_join) cudaEventDestroy(L->ev_join);
  std::free(L->h_table);
  delete L;
  return PCOMOE_OK;
}

pcomoe_status pcomoe_layer_active_set(const pcomoe_layer *L, int32_t cap, int32_t *h_src,
                                      int32_t *h_tgt, float *h_bias, int32_t *count) {
  if (!L || !count || cap < 0) return PCOMOE_ERR_INVALID_ARG;
  *count = L->n_active;
  for (int a = 0; a < L->n_active && a < cap; ++a) {
    if (h_src) h_src[a] = L->h_table[a].src;
    if (h_tgt) h_tgt[a] = L->h_table[a].tgt;
    if (h_bias) h_bias[a] = L->h_table[a].bias;
  }
  return PCOMOE_OK;
}

pcomoe_status pcomoe_workspace_bytes(const pcomoe_layer *L, int32_t max_tokens, size_t *bytes) {
  if (!L || !bytes || max_tokens < 0) return PCOMOE_ERR_INVALID_ARG;
  if ((int64_t)max_tokens * L->cfg.top_k >= (int64_t)1 << 31) return PCOMOE_ERR_SHAPE;
  *bytes = ws_layout(L, max_tokens).total;
  return PCOMOE_OK;
}

pcomoe_status pcomoe_route_paths(const pcomoe_layer *L, int32_t T, const float *d_logits,
                                 const float *d_tgt_logits, int32_t *d_path_src,
                                 int32_t *d_path_tgt, float *d_path_w, void *stream) {
  if (!L) return PCOMOE_ERR_INVALID_ARG;
  if (T < 0) return PCOMOE_ERR_SHAPE;
  if (T == 0) return PCOMOE_OK;
  if (!d_logits || !d_path_src || !d_path_tgt || !d_path_w) return PCOMOE_ERR_INVALID_ARG;
  return launch_route(L, T, d_logits, d_tgt_logits ? d_tgt_logits : d_logits, d_path_src,
                      d_path_tgt, d_path_w, (cudaStream_t)stream);
}

static pcomoe_status check_ws(const pcomoe_layer *L, int32_t T, const void *ws, size_t ws_bytes,
                              WsLayout *lay) {
  if (!ws) return PCOMOE_ERR_WORKSPACE;
  if (((uintptr_t)ws) & 255) return PCOMOE_ERR_WORKSPACE;
  if ((int64_t)T * L->cfg.top_k >= (int64_t)1 << 31) return PCOMOE_ERR_SHAPE;
  *lay = ws_layout(L, T);
  if (lay->total > ws_bytes) return PCOMOE_ERR_WORKSPACE;
  return PCOMOE_OK;
}

static bool groups_ok(const pcomoe_groups *g) {
  return g && g->s1_offsets && g->s1_token && g->path_s1row && g->s2_offsets && g->s2_path &&
         g->s2_s1row && g->s2_token && g->s2_w && g->stats;
}

pcomoe_status pcomoe_build_path_groups(const pcomoe_layer *L, int32_t T, const int32_t *d_path_src,
                                       const int32_t *d_path_tgt, const float *d_path_w,
                                       const pcomoe_groups *out, void *d_workspace, size_t ws_bytes,
                                       void *stream) {
  if (!L || !groups_ok(out)) return PCOMOE_ERR_INVALID_ARG;
  if (T < 0) return PCOMOE_ERR_SHAPE;
  if (T > 0 && (!d_path_src || !d_path_tgt || !d_path_w)) return PCOMOE_ERR_INVALID_ARG;
  WsLayout lay;
  pcomoe_status s = check_ws(L, T, d_workspace, ws_bytes, &lay);
  if (s != PCOMOE_OK) return s;
  return launch_groups(L, T, d_path_src, d_path_tgt, d_path_w, out, (char *)d_workspace, lay,
                       (cudaStream_t)stream);
}

pcomoe_status pcomoe_ffn_forward(const pcomoe_layer *L, int32_t T, const void *d_h,
                                 const void *d_w_gate, const void *d_w_up, const void *d_w_down,
                                 const void *d_wsh_gate, const void *d_wsh_up,
                                 const void *d_wsh_down, const pcomoe_groups *groups, void *d_y,
                                 void *d_workspace, size_t ws_bytes, void *stream) {
  return pcomoe_ffn_forward_stages(L, T, d_h, d_w_gate, d_w_up, d_w_down, d_wsh_gate, d_wsh_up,
                                   d_wsh_down, groups, d_y, d_workspace, ws_bytes, stream, 15);
}

pcomoe_status pcomoe_ffn_forward_stages(const pcomoe_layer *L, int32_t T, const void *d_h,
                                        const void *d_w_gate, const void *d_w_up,
                                        const void *d_w_down, const void *d_wsh_gate,
                                        const void *d_wsh_up, const void *d_wsh_down,
                                        const pcomoe_groups *groups, void *d_y, void *d_workspace,
                                        size_t ws_bytes, void *stream, int32_t stages) {
  if (!L || !groups_ok(groups) || stages < 0 || stages > 15) return PCOMOE_ERR_INVALID_ARG;
  if (T < 0) return PCOMOE_ERR_SHAPE;
  if (T == 0) return PCOMOE_OK;
  if (!d_h || !d_w_gate || !d_w_up || !d_w_down || !d_y) return PCOMOE_ERR_INVALID_ARG;
  if (L->cfg.shared_ffn > 0 && (!d_wsh_gate || !d_wsh_up || !d_wsh_down)) return PCOMOE_ERR_INVALID_ARG;
  WsLayout lay;
  pcomoe_status s = check_ws(L, T, d_workspace, ws_bytes, &lay);
  if (s != PCOMOE_OK) return s;
  const bool tc = L->cfg.ffn_impl >= PCOMOE_FFN_TCGEN05 ||
                  (L->cfg.ffn_impl == PCOMOE_FFN_AUTO && L->tc_ok);
  // a bf16 output is accumulated in fp32 in the workspace and rounded once, after the last addition
  const bool y_bf16 = L->cfg.out_dtype == PCOMOE_BF16;
  float *y_acc = y_bf16 ? reinterpret_cast<float *>((char *)d_workspace + lay.y_acc) : (float *)d_y;
  if (tc)
    s = launch_ffn_tc(L, T, d_h, d_w_gate, d_w_up, d_w_down, d_wsh_gate, d_wsh_up, d_wsh_down,
                      groups, y_acc, (char *)d_workspace, lay, (cudaStream_t)stream, stages);
  else
    s = launch_ffn_simt(L, T, d_h, d_w_gate, d_w_up, d_w_down, d_wsh_gate, d_wsh_up, d_wsh_down,
                        groups, y_acc, (char *)d_workspace, lay, (cudaStream_t)stream, stages);
  if (s == PCOMOE_OK && y_bf16 && (stages & (kStage2Routed | kStage2Shared)))
    s = launch_cast_y(L, T, y_acc, d_y, (cudaStream_t)stream);
  return s;
}

pcomoe_status pcomoe_layer_forward(const pcomoe_layer *L, int32_t T, const float *d_logits,
                                   const float *d_tgt_logits, const void *d_h, const void *d_w_gate,
                                   const void *d_w_up, const void *d_w_down, const void *d_wsh_gate,
                                   const void *d_wsh_up, const void *d_wsh_down, int32_t *d_path_src,
                                   int32_t *d_path_tgt, float *d_path_w, const pcomoe_groups *groups, void *d_y,
                                   void *d_workspace, size_t ws_bytes, void *stream) {
  if (!L || !groups_ok(groups)) return PCOMOE_ERR_INVALID_ARG;
  if (T < 0) return PCOMOE_ERR_SHAPE;
  if (T == 0) return PCOMOE_OK;
  if (!d_logits || !d_h || !d_w_gate || !d_w_up || !d_w_down || !d_path_src || !d_path_tgt || !d_path_w || !d_y)
    return PCOMOE_ERR_INVALID_ARG;
  if (L->cfg.shared_ffn > 0 && (!d_wsh_gate || !d_wsh_up || !d_wsh_down)) return PCOMOE_ERR_INVALID_ARG;
  WsLayout lay;
  pcomoe_status s = check_ws(L, T, d_workspace, ws_bytes, &lay);
  if (s != PCOMOE_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  const bool tc = L->cfg.ffn_impl >= PCOMOE_FFN_TCGEN05 || (L->cfg.ffn_impl == PCOMOE_FFN_AUTO && L->tc_ok);
  // The shared expert's stage 1 needs nothing from routing, grouping and the row gather: on prefill-sized
  // batches it runs on the layer's second stream beside them and joins before stage 2.
  const bool overlap = tc && L->cfg.shared_ffn > 0 && use_cta_pairs(L, T);
  int32_t side_rows = 0;
  if (overlap) {
    // How many tokens of the shared expert the second stream takes: about as many as it can finish while the
    // routing chain runs beside it (the chain runs at roughly half speed then); the rest joins the main stage-1
    // launch, which has the deeper ring and one common tail.  Rough cost model in microseconds.
    const pcomoe_config &c = L->cfg;
    const double route_us = (double)T * L->n_active / 4.5e5;
    const double gather_us = (double)T * c.top_k * 0.7 * c.hidden * 4.0 / 5.5e6;
    const double chain_us = 2.0 * (route_us + 30.0 + gather_us);
    const double side_us_per_token = 4.0 * c.hidden * c.shared_ffn / 1.35e9;
    int64_t rows = (int64_t)(chain_us / side_us_per_token) / 256 * 256;
    if (rows < 256) rows = 256;
    if (rows > T || T - rows < 512) rows = T;
    side_rows = (int32_t)rows;
    PCOMOE_CUDA_TRY(cudaEventRecord(L->ev_fork, st));
    PCOMOE_CUDA_TRY(cudaStreamWaitEvent(L->side_stream, L->ev_fork, 0));
    s = launch_shared_stage1_side(L, T, d_h, d_wsh_gate, d_wsh_up, (char *)d_workspace, lay, L->side_stream, side_rows);
    // the join is recorded whatever happened, so that a stream capture always closes
    PCOMOE_CUDA_TRY(cudaEventRecord(L->ev_join, L->side_stream));
    if (s != PCOMOE_OK) {
      cudaStreamWaitEvent(st, L->ev_join, 0);
      return s;
    }
  }
  const bool y_bf16 = L->cfg.out_dtype == PCOMOE_BF16;
  float *y_acc = y_bf16 ? reinterpret_cast<float *>((char *)d_workspace + lay.y_acc) : (float *)d_y;
  s = launch_route(L, T, d_logits, d_tgt_logits ? d_tgt_logits : d_logits, d_path_src, d_path_tgt, d_path_w, st);
  if (s == PCOMOE_OK)
    s = launch_groups(L, T, d_path_src, d_path_tgt, d_path_w, groups, (char *)d_workspace, lay, st);
  if (s == PCOMOE_OK) {
    if (tc)
      s = launch_ffn_tc(L, T, d_h, d_w_gate, d_w_up, d_w_down, d_wsh_gate, d_wsh_up, d_wsh_down, groups,
                        y_acc, (char *)d_workspace, lay, st,
                        !overlap ? 15 : side_rows < T ? 15 : (kStage1Routed | kStage2Routed | kStage2Shared),
                        overlap ? L->ev_join : nullptr, side_rows);
    else
      s = launch_ffn_simt(L, T, d_h, d_w_gate, d_w_up, d_w_down, d_wsh_gate, d_wsh_up, d_wsh_down, groups,
                          y_acc, (char *)d_workspace, lay, st, 15);
    if (s == PCOMOE_OK && y_bf16) s = launch_cast_y(L, T, y_acc, d_y, st);
  } else if (overlap) {
    cudaStreamWaitEvent(st, L->ev_join, 0);
  }
  return s;
}

pcomoe_status pcomoe_router_logits(const pcomoe_layer *L, int32_t T, const void *d_h, const void *d_w_router,
                                   const void *d_lora_a, const float *d_lora_b, int32_t lora_rank,
                                   float lora_scale, float *d_logits, void *d_workspace, size_t ws_bytes,
                                   void *stream) {
  if (!L || lora_rank < 0) return PCOMOE_ERR_INVALID_ARG;
  if (T < 0) return PCOMOE_ERR_SHAPE;
  if (T == 0) return PCOMOE_OK;
  if (!d_h || !d_w_router || !d_logits) return PCOMOE_ERR_INVALID_ARG;
  if (lora_rank > 0 && (!d_lora_a || !d_lora_b)) return PCOMOE_ERR_INVALID_ARG;
  if (lora_rank > 256) return PCOMOE_ERR_SHAPE;
  WsLayout lay;
  pcomoe_status s = check_ws(L, T, d_workspace, ws_bytes, &lay);
  if (s != PCOMOE_OK) return s;
  DevPlan *plan = reinterpret_cast<DevPlan *>((char *)d_workspace + lay.plan);
  return launch_router(L, T, d_h, d_w_router, d_lora_a, d_lora_b, lora_rank, lora_scale, d_logits,
                       &plan->status_router, (cudaStream_t)stream);
}

pcomoe_status pcomoe_residual_cast(const pcomoe_layer *L, int32_t T, const void *d_h_in, const float *d_y,
                                   void *d_h_out, void *stream) {
  if (!L) return PCOMOE_ERR_INVALID_ARG;
  if (T < 0) return PCOMOE_ERR_SHAPE;
  if (T == 0) return PCOMOE_OK;
  if (!d_h_in || !d_y || !d_h_out) return PCOMOE_ERR_INVALID_ARG;
  if (L->cfg.out_dtype != PCOMOE_FP32) return PCOMOE_ERR_UNSUPPORTED;   // d_y is read as fp32
  return launch_residual_cast(L, T, d_h_in, d_y, d_h_out, (cudaStream_t)stream);
}

pcomoe_status pcomoe_device_status(const void *d_workspace, void *stream) {
  if (!d_workspace) return PCOMOE_ERR_WORKSPACE;
  DevPlan plan;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return PCOMOE_ERR_CUDA;
  if (cudaMemcpy(&plan, d_workspace, sizeof(DevPlan), cudaMemcpyDeviceToHost) != cudaSuccess)
    return PCOMOE_ERR_CUDA;
  const int32_t st = plan.status ? plan.status : plan.status_router;
  if (plan.status_router != 0) {   // the router's word is sticky: reading it clears it
    if (cudaMemset((char *)const_cast<void *>(d_workspace) + offsetof(DevPlan, status_router), 0, sizeof(int32_t)) !=
        cudaSuccess)
      return PCOMOE_ERR_CUDA;
  }
  if (st < 0 || st > PCOMOE_ERR_INDEX) return PCOMOE_ERR_CUDA;
  return (pcomoe_status)st;
}

pcomoe_status pcomoe_set_wait_limit_us(uint32_t limit_us) {
  if (limit_us == 0) limit_us = 2000000u;
  if (limit_us > 60000000u) return PCOMOE_ERR_INVALID_ARG;
  g_wait_limit_ns.store((uint64_t)limit_us * 1000ull, std::memory_order_relaxed);
  return PCOMOE_OK;
}

pcomoe_status pcomoe_selftest_wait_timeout(void *d_workspace, void *stream) {
  if (!d_workspace) return PCOMOE_ERR_WORKSPACE;
  if (((uintptr_t)d_workspace) & 255) return PCOMOE_ERR_WORKSPACE;
  DevPlan *plan = reinterpret_cast<DevPlan *>(d_workspace);
  return launch_wait_probe(&plan->status, (cudaStream_t)stream);
}

int64_t pcomoe_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char *pcomoe_status_string(pcomoe_status s) {
  switch (s) {
    case PCOMOE_OK: return "ok";
    case PCOMOE_ERR_INVALID_ARG: return "invalid argument";
    case PCOMOE_ERR_SHAPE: return "shape out of range";
    case PCOMOE_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case PCOMOE_ERR_UNSUPPORTED: return "unsupported size or dtype";
    case PCOMOE_ERR_CUDA: return "CUDA call failed";
    case PCOMOE_ERR_TIMEOUT: return "device wait timed out";
    case PCOMOE_ERR_INDEX: return "device index out of range";
  }
  return "unknown status";
}

}  // extern "C"
