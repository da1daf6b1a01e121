#include "common.cuh"
bool dc_conv_tc_supported(int, int, int, const dc_geom *) { return false; }
dc_status dc_launch_conv_tc(const void *, int, int, int, const dc_geom *, const void *, const float *, dc_act,
                            const void *, void *, void *, cudaStream_t) { return DC_ERR_UNSUPPORTED; }
