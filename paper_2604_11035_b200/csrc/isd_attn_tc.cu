// placeholder until the tensor-core kernel lands
#include "isd_internal.cuh"
int isd_attn_tc_create(isd_ctx*) { return ISD_OK; }
void isd_attn_tc_destroy(isd_ctx*) {}
int isd_launch_attn_tc(isd_ctx*, const isd_batch_state*, const void*, const void*, const void*, void*, void*,
                       void*, float*, cudaStream_t) { return ISD_ERR_UNSUPPORTED; }
