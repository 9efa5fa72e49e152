// Decode attention for callers that cannot provide or allocate a workspace.
//
// Who needs this: an inference engine that claims all device memory for its own pool at start-up
// and hands the library no scratch buffer; a plug-in loaded into such an engine; a serving loop
// that must not call cudaMalloc because the call synchronises the device and its latency is
// unbounded.  For them the scratch that novakv_decode_attention takes as `workspace` lives here, in
// a fixed array in the library's own device image.
//
// Consequences the caller must know:
//   - the array exists once per GPU that loads the library, from load until the process exits;
//   - it holds NOVAKV_NOALLOC_SCRATCH_BYTES, so batches whose workspace would be larger are refused;
//   - every call on a device uses the same array: two calls that overlap on the GPU (different
//     streams, or different contexts on one device) race on it.  Calls on one stream are ordered and
//     safe.  The decode kernels write every scratch word before reading it, so nothing has to be
//     cleared between calls and the previous call's contents are harmless;
//   - the first call on each device looks up the array's device address (a synchronous runtime
//     query); make that first call before starting any stream capture.
#include "novakv_internal.cuh"

// The scratch itself.  In host code this name is only a handle for the runtime, not an address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOVAKV_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int MAX_DEVICES = 64;
void* g_scratch_ptr[MAX_DEVICES] = {nullptr};

// Device address of the array on `device` (which must be current); looked up once per device.
novakv_status scratch_address(int device, void** out) {
    if (device < 0 || device >= MAX_DEVICES) return NOVAKV_EINVAL;
    if (g_scratch_ptr[device] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) return NOVAKV_ECUDA;
        g_scratch_ptr[device] = p;
    }
    *out = g_scratch_ptr[device];
    return NOVAKV_OK;
}

}  // namespace

extern "C" novakv_status novakv_decode_attention_noalloc(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, const int32_t* seq_lens, int batch, float sm_scale, void* out, int out_is_fp32,
    novakv_stream stream) {
    if (!ctx) return NOVAKV_EINVAL;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return NOVAKV_EINVAL;
    if (!ctx->layers[layer].loaded) return NOVAKV_ENOCALIB;
    if (batch < 0) return NOVAKV_EINVAL;
    if (batch == 0) return NOVAKV_OK;
    if (!q || !k_pages || !v_pages || !page_table || !seq_lens || !out) return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= 0) return NOVAKV_EPAGE;
    if (((uintptr_t)k_pages & 15) || ((uintptr_t)v_pages & 15)) return NOVAKV_EINVAL;
    if (!(sm_scale == sm_scale)) return NOVAKV_EINVAL;
    // the batch must fit the fixed array
    const size_t need = novakv_decode_ws_bytes(ctx, batch);
    if (need > (size_t)NOVAKV_NOALLOC_SCRATCH_BYTES) return NOVAKV_EWORKSPACE;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    void* scratch = nullptr;
    novakv_status st = scratch_address(ctx->cfg.device, &scratch);
    if (st != NOVAKV_OK) return st;
    // per-kernel event timing creates events on demand; this entry point must not, so it runs with
    // the timing hooks off whatever the context's setting is
    const bool prof = ctx->profile;
    ctx->profile = false;
    st = novakv_launch_decode(ctx, ctx->layers[layer], (const __nv_bfloat16*)q, k_pages, v_pages, n_pages,
                              page_table, max_pages_per_seq, seq_lens, batch, sm_scale, out, out_is_fp32,
                              scratch, need, (cudaStream_t)stream);
    ctx->profile = prof;
    return st;
}
