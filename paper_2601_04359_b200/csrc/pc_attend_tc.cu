// placeholder until the tcgen05 kernel lands
#include "pc_common.cuh"
pc_status pc_attend_tc_scratch(const pc_layer_desc *d, int sm_count, size_t *k_rot_rows, size_t *part_o_floats,
                               size_t *part_ml_floats) {
    *k_rot_rows = 1; *part_o_floats = 1; *part_ml_floats = 1;
    return PC_OK;
}
pc_status pc_launch_attend_tc(pc_ctx *ctx, int n_seg, const pc_segment *segs, const void *q, const int32_t *q_pos,
                              int32_t n_q, void *out, float *lse, cudaStream_t stream) {
    return pc_launch_attend_simt(ctx, n_seg, segs, q, q_pos, n_q, out, lse, stream);
}
