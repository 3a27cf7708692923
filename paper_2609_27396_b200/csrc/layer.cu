// Full backbone block around the all-boundary attention.
#include "layer.cuh"

namespace dpara {

size_t layer_workspace_bytes(const dpara_shape *, const dpara_layer_io *) { return 0; }

dpara_status launch_layer(const dpara_shape *, const dpara_attn_io *, const dpara_layer_io *, void *, int32_t *, cudaStream_t) {
  return DPARA_ERR_UNSUPPORTED;
}

}  // namespace dpara
