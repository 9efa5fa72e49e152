// Uncompressed bf16 paged decode attention (comparator for the compression speed-up).
#include "novakv_internal.cuh"

size_t novakv_bf16_ws_bytes(const novakv_ctx* ctx, int batch, int max_pages_per_seq) {
    (void)ctx; (void)batch; (void)max_pages_per_seq;
    return 256;
}

novakv_status novakv_launch_bf16_decode(novakv_ctx* ctx, const __nv_bfloat16* q,
    const __nv_bfloat16* k_pages, const __nv_bfloat16* v_pages, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, const int32_t* seq_lens, int batch,
    float sm_scale, int window, void* out, int out_is_fp32, void* workspace, size_t workspace_bytes,
    cudaStream_t stream) {
    return NOVAKV_ESHAPE;
}
