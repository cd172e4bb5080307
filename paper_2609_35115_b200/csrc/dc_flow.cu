// placeholder until the bf16 flow decoder lands
#include "dc_internal.h"
namespace dc {
dc_status flow_model_create(const dc_config&, const float*, FlowModel**) { set_error("flow decoder not built"); return DC_ERR_CONFIG; }
void flow_model_destroy(FlowModel*) {}
dc_status flow_state_open(FlowModel*, FlowState**) { return DC_ERR_CONFIG; }
void flow_state_buffers(const FlowState*, DevBuf*, int, int* n) { *n = 0; }
dc_status flow_state_reset(FlowModel*, FlowState*, cudaStream_t) { return DC_ERR_CONFIG; }
void flow_state_close(FlowState*) {}
dc_status flow_decode(FlowModel*, int, FlowState* const*, const float* const*, const int*, float* const*, cudaStream_t, int*) { return DC_ERR_CONFIG; }
}
