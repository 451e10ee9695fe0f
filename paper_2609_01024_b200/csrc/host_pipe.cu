// pcomoe_host_pipe: the whole hot path for batches that live in host memory.  Per batch: host->device copies of
// logits and hidden states on a copy-in stream, pcomoe_layer_forward on a compute stream, device->host copy of y
// on a copy-out stream, ordered by events; the input and output device buffers exist in several slots so that
// the copies of neighbouring batches overlap the kernels.  Everything the kernels share between batches (path
// and group arrays, workspace) exists once, because the compute stream runs the batches one after another.
#include <new>

#include "common.cuh"

using namespace pcomoe;

namespace {

constexpr int kMaxSlots = 4;

struct Slot {
  float *d_logits = nullptr, *d_tgt_logits = nullptr;
  void *d_h = nullptr, *d_y = nullptr;
  cudaEvent_t ev_in = nullptr, ev_done = nullptr, ev_out = nullptr;
  bool used = false;
};

// Keeps the first device-side error of any batch: the layer's status word is cleared by every grouping step.
__global__ void latch_status_kernel(const DevPlan *plan, int32_t *sticky) {
  pdl_grid_wait();
  if (threadIdx.x == 0) {
    const int32_t st = plan->status ? plan->status : plan->status_router;
    if (st != 0 && *sticky == 0) *sticky = st;
  }
}

size_t up256(size_t x) { return (x + 255) & ~size_t(255); }

}  // namespace

struct pcomoe_host_pipe {
  const pcomoe_layer *L = nullptr;
  int32_t max_tokens = 0, slots = 0;
  const void *wg = nullptr, *wu = nullptr, *wd = nullptr, *sg = nullptr, *su = nullptr, *sd = nullptr;
  cudaStream_t s_in = nullptr, s_main = nullptr, s_out = nullptr;
  Slot slot[kMaxSlots];
  int32_t *d_src = nullptr, *d_tgt = nullptr;
  float *d_w = nullptr;
  pcomoe_groups g = {};
  char *ws = nullptr;
  size_t ws_bytes = 0;
  int32_t *d_sticky = nullptr;
  char *arena = nullptr;
  int64_t step = 0;
};

extern "C" {

pcomoe_status pcomoe_host_pipe_destroy(pcomoe_host_pipe *P) {
  if (!P) return PCOMOE_ERR_INVALID_ARG;
  if (P->s_in) cudaStreamSynchronize(P->s_in);
  if (P->s_main) cudaStreamSynchronize(P->s_main);
  if (P->s_out) cudaStreamSynchronize(P->s_out);
  for (int i = 0; i < kMaxSlots; ++i) {
    if (P->slot[i].ev_in) cudaEventDestroy(P->slot[i].ev_in);
    if (P->slot[i].ev_done) cudaEventDestroy(P->slot[i].ev_done);
    if (P->slot[i].ev_out) cudaEventDestroy(P->slot[i].ev_out);
  }
  if (P->s_in) cudaStreamDestroy(P->s_in);
  if (P->s_main) cudaStreamDestroy(P->s_main);
  if (P->s_out) cudaStreamDestroy(P->s_out);
  if (P->arena) cudaFree(P->arena);
  delete P;
  return PCOMOE_OK;
}

pcomoe_status pcomoe_host_pipe_create(const pcomoe_layer *L, int32_t max_tokens, int32_t slots,
                                      const void *d_w_gate, const void *d_w_up, const void *d_w_down,
                                      const void *d_wsh_gate, const void *d_wsh_up, const void *d_wsh_down,
                                      pcomoe_host_pipe **out) {
  if (!L || !out || !d_w_gate || !d_w_up || !d_w_down) return PCOMOE_ERR_INVALID_ARG;
  if (L->cfg.shared_ffn > 0 && (!d_wsh_gate || !d_wsh_up || !d_wsh_down)) return PCOMOE_ERR_INVALID_ARG;
  if (max_tokens <= 0 || slots < 1 || slots > kMaxSlots) return PCOMOE_ERR_SHAPE;
  if ((int64_t)max_tokens * L->cfg.top_k >= (int64_t)1 << 31) return PCOMOE_ERR_SHAPE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return PCOMOE_ERR_CUDA;
  if (dev != L->device) return PCOMOE_ERR_INVALID_ARG;
  pcomoe_host_pipe *P = new (std::nothrow) pcomoe_host_pipe();
  if (!P) return PCOMOE_ERR_CUDA;
  P->L = L; P->max_tokens = max_tokens; P->slots = slots;
  P->wg = d_w_gate; P->wu = d_w_up; P->wd = d_w_down; P->sg = d_wsh_gate; P->su = d_wsh_up; P->sd = d_wsh_down;
  const pcomoe_config &c = L->cfg;
  const size_t T = (size_t)max_tokens, n = (size_t)c.n_experts, K = (size_t)c.top_k, H = (size_t)c.hidden;
  const size_t PK = T * K;
  const size_t b_logits = up256(T * n * 4), b_h = up256(T * H * dtype_size(c.in_dtype)),
               b_y = up256(T * H * dtype_size(c.out_dtype));
  P->ws_bytes = ws_layout(L, max_tokens).total;
  size_t total = 256 + (size_t)slots * (2 * b_logits + b_h + b_y) + 3 * up256(PK * 4) +
                 2 * up256((n + 1) * 4) + 6 * up256(PK * 4) + 256 + up256(P->ws_bytes);
  cudaError_t e = cudaMalloc((void **)&P->arena, total);
  if (e == cudaSuccess) e = cudaMemset(P->arena, 0, 512);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&P->s_in, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&P->s_main, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&P->s_out, cudaStreamNonBlocking);
  for (int i = 0; i < slots && e == cudaSuccess; ++i) {
    e = cudaEventCreateWithFlags(&P->slot[i].ev_in, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&P->slot[i].ev_done, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&P->slot[i].ev_out, cudaEventDisableTiming);
  }
  if (e != cudaSuccess) {
    pcomoe_host_pipe_destroy(P);
    return PCOMOE_ERR_CUDA;
  }
  char *p = P->arena;
  auto take = [&](size_t bytes) { char *q = p; p += bytes; return q; };
  P->d_sticky = reinterpret_cast<int32_t *>(take(256));
  for (int i = 0; i < slots; ++i) {
    P->slot[i].d_logits = reinterpret_cast<float *>(take(b_logits));
    P->slot[i].d_tgt_logits = reinterpret_cast<float *>(take(b_logits));
    P->slot[i].d_h = take(b_h);
    P->slot[i].d_y = take(b_y);
  }
  P->d_src = reinterpret_cast<int32_t *>(take(up256(PK * 4)));
  P->d_tgt = reinterpret_cast<int32_t *>(take(up256(PK * 4)));
  P->d_w = reinterpret_cast<float *>(take(up256(PK * 4)));
  P->g.s1_offsets = reinterpret_cast<int32_t *>(take(up256((n + 1) * 4)));
  P->g.s2_offsets = reinterpret_cast<int32_t *>(take(up256((n + 1) * 4)));
  P->g.s1_token = reinterpret_cast<int32_t *>(take(up256(PK * 4)));
  P->g.path_s1row = reinterpret_cast<int32_t *>(take(up256(PK * 4)));
  P->g.s2_path = reinterpret_cast<int32_t *>(take(up256(PK * 4)));
  P->g.s2_s1row = reinterpret_cast<int32_t *>(take(up256(PK * 4)));
  P->g.s2_token = reinterpret_cast<int32_t *>(take(up256(PK * 4)));
  P->g.s2_w = reinterpret_cast<float *>(take(up256(PK * 4)));
  P->g.stats = reinterpret_cast<int32_t *>(take(256));
  P->ws = take(up256(P->ws_bytes));   // arena is 256-byte aligned and every section is a multiple of 256
  *out = P;
  return PCOMOE_OK;
}

pcomoe_status pcomoe_host_pipe_submit(pcomoe_host_pipe *P, int32_t T, const float *h_logits,
                                      const float *h_tgt_logits, const void *h_hidden, void *h_y) {
  if (!P) return PCOMOE_ERR_INVALID_ARG;
  if (T < 0 || T > P->max_tokens) return PCOMOE_ERR_SHAPE;
  if (T == 0) return PCOMOE_OK;
  if (!h_logits || !h_hidden || !h_y) return PCOMOE_ERR_INVALID_ARG;
  const pcomoe_layer *L = P->L;
  const pcomoe_config &c = L->cfg;
  Slot &S = P->slot[P->step % P->slots];
  const size_t b_logits = (size_t)T * c.n_experts * 4, b_h = (size_t)T * c.hidden * dtype_size(c.in_dtype),
               b_y = (size_t)T * c.hidden * dtype_size(c.out_dtype);
  if (S.used) {
    PCOMOE_CUDA_TRY(cudaStreamWaitEvent(P->s_in, S.ev_done, 0));    // the slot's inputs have been consumed
    PCOMOE_CUDA_TRY(cudaStreamWaitEvent(P->s_main, S.ev_out, 0));   // the slot's y has been copied out
  }
  PCOMOE_CUDA_TRY(cudaMemcpyAsync(S.d_logits, h_logits, b_logits, cudaMemcpyHostToDevice, P->s_in));
  if (h_tgt_logits)
    PCOMOE_CUDA_TRY(cudaMemcpyAsync(S.d_tgt_logits, h_tgt_logits, b_logits, cudaMemcpyHostToDevice, P->s_in));
  PCOMOE_CUDA_TRY(cudaMemcpyAsync(S.d_h, h_hidden, b_h, cudaMemcpyHostToDevice, P->s_in));
  PCOMOE_CUDA_TRY(cudaEventRecord(S.ev_in, P->s_in));
  PCOMOE_CUDA_TRY(cudaStreamWaitEvent(P->s_main, S.ev_in, 0));
  const pcomoe_status st = pcomoe_layer_forward(L, T, S.d_logits, h_tgt_logits ? S.d_tgt_logits : nullptr, S.d_h, P->wg,
                                                P->wu, P->wd, P->sg, P->su, P->sd, P->d_src, P->d_tgt, P->d_w, &P->g,
                                                S.d_y, P->ws, P->ws_bytes, P->s_main);
  if (st == PCOMOE_OK) {
    PCOMOE_CUDA_TRY(launch_pdl(latch_status_kernel, dim3(1), dim3(32), 0, P->s_main,
                               reinterpret_cast<const DevPlan *>(P->ws), P->d_sticky));
    count_launch();
  }
  PCOMOE_CUDA_TRY(cudaEventRecord(S.ev_done, P->s_main));
  PCOMOE_CUDA_TRY(cudaStreamWaitEvent(P->s_out, S.ev_done, 0));
  if (st == PCOMOE_OK) PCOMOE_CUDA_TRY(cudaMemcpyAsync(h_y, S.d_y, b_y, cudaMemcpyDeviceToHost, P->s_out));
  PCOMOE_CUDA_TRY(cudaEventRecord(S.ev_out, P->s_out));
  S.used = true;
  ++P->step;
  return st;
}

pcomoe_status pcomoe_host_pipe_wait(pcomoe_host_pipe *P) {
  if (!P) return PCOMOE_ERR_INVALID_ARG;
  PCOMOE_CUDA_TRY(cudaStreamSynchronize(P->s_in));
  PCOMOE_CUDA_TRY(cudaStreamSynchronize(P->s_main));
  PCOMOE_CUDA_TRY(cudaStreamSynchronize(P->s_out));
  int32_t st = 0;
  PCOMOE_CUDA_TRY(cudaMemcpy(&st, P->d_sticky, sizeof(st), cudaMemcpyDeviceToHost));
  if (st != 0) {
    PCOMOE_CUDA_TRY(cudaMemset(P->d_sticky, 0, sizeof(st)));
    // the router's word is sticky as well: clear it with the report
    PCOMOE_CUDA_TRY(cudaMemset(P->ws + offsetof(DevPlan, status_router), 0, sizeof(int32_t)));
  }
  if (st < 0 || st > PCOMOE_ERR_INDEX) return PCOMOE_ERR_CUDA;
  return (pcomoe_status)st;
}

pcomoe_status pcomoe_host_pipe_arrays(const pcomoe_host_pipe *P, pcomoe_groups *groups, int32_t **d_path_src,
                                      int32_t **d_path_tgt, float **d_path_w) {
  if (!P) return PCOMOE_ERR_INVALID_ARG;
  if (groups) *groups = P->g;
  if (d_path_src) *d_path_src = P->d_src;
  if (d_path_tgt) *d_path_tgt = P->d_tgt;
  if (d_path_w) *d_path_w = P->d_w;
  return PCOMOE_OK;
}

}  // extern "C"
