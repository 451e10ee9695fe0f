#include "common.cuh"
namespace pcomoe {
pcomoe_status launch_ffn_tc(const pcomoe_layer *L, int32_t T, const void *h, const void *wg,
                            const void *wu, const void *wd, const void *sg, const void *su,
                            const void *sd, const pcomoe_groups *g, float *y, char *ws,
                            const WsLayout &lay, cudaStream_t st) {
  return PCOMOE_ERR_UNSUPPORTED;
}
}  // namespace pcomoe
