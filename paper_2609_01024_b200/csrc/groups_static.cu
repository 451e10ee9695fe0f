// pcomoe_build_path_groups_static: the grouping step for callers that cannot hand over a workspace.
//
// pcomoe_build_path_groups needs device scratch (per-block histograms, tile prefixes, gather maps) and
// takes it from a caller-allocated workspace.  A caller that has no way to obtain device memory at the
// point of the call - a routing plug-in loaded into a serving process whose engine has already claimed
// the whole device for its own pools, or code running where any allocation (and the device-wide
// synchronisation a cudaMalloc/cudaFree implies) is forbidden by the host application - cannot provide
// one.  Here the scratch is a fixed array in the library's own device image instead.
#include <mutex>

#include "common.cuh"

namespace pcomoe {
namespace {

// Scratch of the grouping kernels.  Lives in every device that loads the library until the process exits.
static __device__ __align__(256) unsigned char g_group_scratch[PCOMOE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
char *g_scratch_addr[kMaxDevices] = {nullptr};   // device address of g_group_scratch, per device ordinal

// In host code `g_group_scratch` is only a handle for the symbol, never an address a kernel may use:
// the device address has to be asked for, with the owning device current.
pcomoe_status scratch_for_current_device(int dev, char **out) {
  if (dev < 0 || dev >= kMaxDevices) return PCOMOE_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_group_scratch) != cudaSuccess || !p) return PCOMOE_ERR_CUDA;
    g_scratch_addr[dev] = static_cast<char *>(p);
  }
  *out = g_scratch_addr[dev];
  return PCOMOE_OK;
}

}  // namespace
}  // namespace pcomoe

using namespace pcomoe;

extern "C" pcomoe_status pcomoe_build_path_groups_static(const pcomoe_layer *L, int32_t T,
                                                         const int32_t *d_path_src,
                                                         const int32_t *d_path_tgt,
                                                         const float *d_path_w,
                                                         const pcomoe_groups *out, void *stream) {
  if (!L || !out || !out->s1_offsets || !out->s1_token || !out->path_s1row || !out->s2_offsets ||
      !out->s2_path || !out->s2_s1row || !out->s2_token || !out->s2_w || !out->stats)
    return PCOMOE_ERR_INVALID_ARG;
  if (T < 0) return PCOMOE_ERR_SHAPE;
  if (T > 0 && (!d_path_src || !d_path_tgt || !d_path_w)) return PCOMOE_ERR_INVALID_ARG;
  if ((int64_t)T * L->cfg.top_k >= (int64_t)1 << 31) return PCOMOE_ERR_SHAPE;
  if (L->cfg.target_reuse) return PCOMOE_ERR_UNSUPPORTED;   // that mode keeps a per-path array beyond the scratch
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return PCOMOE_ERR_CUDA;
  if (dev != L->device) return PCOMOE_ERR_INVALID_ARG;   // the layer's table lives on its own device
  // the grouping kernels touch only the sections of the workspace layout that precede the intermediates
  const WsLayout lay = ws_layout(L, T);
  if (lay.u > (size_t)PCOMOE_STATIC_SCRATCH_BYTES) return PCOMOE_ERR_SHAPE;
  char *scratch = nullptr;
  const pcomoe_status s = scratch_for_current_device(dev, &scratch);
  if (s != PCOMOE_OK) return s;
  // launch_groups zero-fills the header and rewrites every entry it later reads, so nothing of an earlier
  // call survives
  return launch_groups(L, T, d_path_src, d_path_tgt, d_path_w, out, scratch, lay, (cudaStream_t)stream);
}
