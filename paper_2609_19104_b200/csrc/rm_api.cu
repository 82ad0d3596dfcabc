// C-ABI entry points: argument validation and dispatch.  Every step of the path runs in the library's kernels.
#include <new>

#include "rm_common.cuh"

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline bool all_aligned(std::initializer_list<const void*> ps) {
    for (const void* p : ps)
        if (p && !rm_aligned16(p)) return false;
    return true;
}

}  // namespace

extern "C" {

int rm_create(rm_ctx** out, const rm_model_desc* desc) {
    if (!out) return RM_ERR_INVALID_ARG;
    *out = nullptr;
    if (!desc) return RM_ERR_INVALID_ARG;
    if (desc->L < 1 || desc->H < 64 || desc->I < 1 || desc->T_max < 1 || desc->B_max < 1) return RM_ERR_INVALID_ARG;
    if (desc->H % 64 != 0) return RM_ERR_SHAPE;
    if (desc->act != RM_ACT_GELU_TANH) return RM_ERR_UNSUPPORTED;
    rm_ctx* c = new (std::nothrow) rm_ctx();
    if (!c) return RM_ERR_CUDA;
    c->desc = *desc;
    c->g.L = desc->L;
    c->g.H = desc->H;
    c->g.I = desc->I;
    c->g.Hs = desc->H / RM_NS;
    c->launches = 0;
    c->d_status = nullptr;
    cudaDeviceProp prop;
    if (cudaGetDevice(&c->device) != cudaSuccess || cudaGetDeviceProperties(&prop, c->device) != cudaSuccess ||
        cudaMalloc(&c->d_status, 256) != cudaSuccess || cudaMemset(c->d_status, 0, 256) != cudaSuccess) {
        if (c->d_status) cudaFree(c->d_status);
        delete c;
        return RM_ERR_CUDA;
    }
    c->sm_count = prop.multiProcessorCount;
    *out = c;
    return RM_OK;
}

int rm_destroy(rm_ctx* ctx) {
    if (!ctx) return RM_ERR_INVALID_ARG;
    cudaFree(ctx->d_status);
    delete ctx;
    return RM_OK;
}

size_t rm_packed_layer_bytes(const rm_ctx* ctx) {
    return ctx ? (size_t)ctx->g.I * 3 * ctx->g.H * sizeof(__nv_bfloat16) : 0;
}

size_t rm_workspace_bytes(const rm_ctx* ctx, int B, int T) {
    if (!ctx || B < 1 || T < 1) return 0;
    // layer scratch + two residual-stream buffers (ping-pong between layers, and the host variant's staging)
    size_t r_bytes = align_up((size_t)B * T * ctx->g.H * sizeof(float), 256);
    return rm_ref_workspace_bytes(ctx, B, T) + 2 * r_bytes;
}

int rm_pack_weights(rm_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, void* packed_out,
                    float* down_colnorm, rm_stream_t stream) {
    if (!ctx || !Wg || !Wu || !Wd || !packed_out) return RM_ERR_INVALID_ARG;
    if (!all_aligned({Wg, Wu, Wd, packed_out, down_colnorm})) return RM_ERR_ALIGN;
    return rm_launch_pack(ctx, Wg, Wu, Wd, packed_out, down_colnorm, static_cast<cudaStream_t>(stream));
}

int rm_mask_compact(rm_ctx* ctx, const rm_mask_src* src, int32_t* idx_out, int32_t* count_out, int64_t stride,
                    rm_stream_t stream) {
    if (!ctx || !src || !idx_out || !count_out || !src->records) return RM_ERR_INVALID_ARG;
    if (src->n_lists < 0 || src->I < 1 || stride < 1) return RM_ERR_INVALID_ARG;
    if (src->n_records < 1 || src->n_records > 16) return RM_ERR_INVALID_ARG;
    if (src->kind == RM_SRC_BOOL_U8) {
        if (src->reduce != RM_REDUCE_NONE) return RM_ERR_INVALID_ARG;
    } else if (src->kind == RM_SRC_SCORE_F32) {
        if (src->reduce != RM_REDUCE_THRESHOLD && src->reduce != RM_REDUCE_TOPK && src->reduce != RM_REDUCE_GROUP)
            return RM_ERR_INVALID_ARG;
    } else {
        return RM_ERR_INVALID_ARG;
    }
    if (src->reduce != RM_REDUCE_GROUP && (src->min_votes < 1 || src->min_votes > src->n_records))
        return RM_ERR_INVALID_ARG;
    if ((src->reduce == RM_REDUCE_TOPK || src->reduce == RM_REDUCE_GROUP) && src->k < 0) return RM_ERR_INVALID_ARG;
    for (int w = 0; w < src->n_records; ++w) {
        if (!src->records[w]) return RM_ERR_INVALID_ARG;
        if (!rm_aligned16(src->records[w])) return RM_ERR_ALIGN;
    }
    if (!all_aligned({idx_out, src->scale})) return RM_ERR_ALIGN;
    if (src->scale && src->kind != RM_SRC_SCORE_F32) return RM_ERR_INVALID_ARG;
    return rm_launch_mask_compact(ctx, src, idx_out, count_out, stride, static_cast<cudaStream_t>(stream));
}

int rm_sparse_mlp(rm_ctx* ctx, const void* packed_layer, const void* x, const float* residual, const int32_t* idx,
                  const int32_t* count_dev, float* y, float* record_out, const float* record_scale, int T, void* ws,
                  size_t ws_bytes, rm_stream_t stream) {
    if (!ctx || !packed_layer || !x || !y || T < 0) return RM_ERR_INVALID_ARG;
    if (idx && !count_dev) return RM_ERR_INVALID_ARG;
    if (idx && record_out) return RM_ERR_INVALID_ARG;       // records are emitted by dense passes only
    if (T > ctx->desc.T_max) return RM_ERR_SHAPE;
    if (!all_aligned({packed_layer, x, residual, idx, y, record_out, record_scale, ws})) return RM_ERR_ALIGN;
    if (T == 0) return RM_OK;
    if (!ws || ws_bytes < rm_workspace_bytes(ctx, 1, T)) return RM_ERR_WORKSPACE;
    rm_layer_args a{};
    a.packed = static_cast<const __nv_bfloat16*>(packed_layer);
    a.x = static_cast<const __nv_bfloat16*>(x);
    a.r_in = residual;
    a.r_out = y;
    a.idx = idx;
    a.count = count_dev;
    a.idx_stride = ctx->g.I;
    a.list_cap = ctx->g.I;
    a.count_stride = 1;
    a.record = record_out;
    a.record_stride = ctx->g.I;
    a.record_scale = record_scale;
    a.B = 1;
    a.T = T;
    return rm_launch_layer_ref(ctx, a, ws, static_cast<cudaStream_t>(stream));
}

static int step_device(rm_ctx* ctx, const void* const* packed_layers, const float* r_in, const int32_t* idx,
                       const int32_t* count_dev, int64_t stride, float* r_out, float* records_out,
                       const float* record_scale, int B, int T, void* ws, cudaStream_t s) {
    const rm_geom& g = ctx->g;
    char* layer_ws = static_cast<char*>(ws);
    const float* cur = r_in;
    for (int l = 0; l < g.L; ++l) {
        rm_layer_args a{};
        a.packed = static_cast<const __nv_bfloat16*>(packed_layers[l]);
        a.x = nullptr;
        a.r_in = cur;
        a.r_out = r_out;                                   // in place after the first layer
        a.idx = idx ? idx + (size_t)l * stride : nullptr;
        a.count = idx ? count_dev + l : nullptr;
        a.idx_stride = (int64_t)g.L * stride;
        a.list_cap = stride;
        a.count_stride = g.L;
        a.record = records_out ? records_out + (size_t)l * g.I : nullptr;
        a.record_stride = (int64_t)g.L * g.I;
        a.record_scale = record_scale ? record_scale + (size_t)l * g.I : nullptr;
        a.B = B;
        a.T = T;
        int rc = rm_launch_layer_ref(ctx, a, layer_ws, s);
        if (rc != RM_OK) return rc;
        cur = r_out;
    }
    return RM_OK;
}

int rm_action_expert_step(rm_ctx* ctx, const void* const* packed_layers, const float* r_in, const int32_t* idx,
                          const int32_t* count_dev, int64_t stride, float* r_out, float* records_out,
                          const float* record_scale, int B, int T, void* ws, size_t ws_bytes, rm_stream_t stream) {
    if (!ctx || !packed_layers || !r_in || !r_out || B < 0 || T < 0) return RM_ERR_INVALID_ARG;
    if (idx && (!count_dev || stride < 1)) return RM_ERR_INVALID_ARG;
    if (idx && records_out) return RM_ERR_INVALID_ARG;
    if (B > ctx->desc.B_max || T > ctx->desc.T_max) return RM_ERR_SHAPE;
    for (int l = 0; l < ctx->g.L; ++l) {
        if (!packed_layers[l]) return RM_ERR_INVALID_ARG;
        if (!rm_aligned16(packed_layers[l])) return RM_ERR_ALIGN;
    }
    if (!all_aligned({r_in, idx, r_out, records_out, record_scale, ws})) return RM_ERR_ALIGN;
    if (idx && (stride % 4) != 0) return RM_ERR_ALIGN;       // every list must start 16-byte aligned
    if (B == 0 || T == 0) return RM_OK;
    if (!ws || ws_bytes < rm_workspace_bytes(ctx, B, T)) return RM_ERR_WORKSPACE;
    return step_device(ctx, packed_layers, r_in, idx, count_dev, stride, r_out, records_out, record_scale, B, T, ws,
                       static_cast<cudaStream_t>(stream));
}

int rm_action_expert_step_host(rm_ctx* ctx, const void* const* packed_layers, const float* r_in_host,
                               const int32_t* idx, const int32_t* count_dev, int64_t stride, float* r_out_host, int B,
                               int T, void* ws, size_t ws_bytes, rm_stream_t stream) {
    if (!ctx || !packed_layers || !r_in_host || !r_out_host || B < 0 || T < 0) return RM_ERR_INVALID_ARG;
    if (idx && (!count_dev || stride < 1)) return RM_ERR_INVALID_ARG;
    if (B > ctx->desc.B_max || T > ctx->desc.T_max) return RM_ERR_SHAPE;
    for (int l = 0; l < ctx->g.L; ++l) {
        if (!packed_layers[l]) return RM_ERR_INVALID_ARG;
        if (!rm_aligned16(packed_layers[l])) return RM_ERR_ALIGN;
    }
    if (!all_aligned({idx, ws})) return RM_ERR_ALIGN;
    if (idx && (stride % 4) != 0) return RM_ERR_ALIGN;
    if (B == 0 || T == 0) return RM_OK;
    if (!ws || ws_bytes < rm_workspace_bytes(ctx, B, T)) return RM_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t n_bytes = (size_t)B * T * ctx->g.H * sizeof(float);
    // the last residual-stream buffer of the workspace is the staging copy
    float* stage = reinterpret_cast<float*>(static_cast<char*>(ws) + rm_workspace_bytes(ctx, B, T) -
                                            align_up(n_bytes, 256));
    RM_CUDA_TRY(cudaMemcpyAsync(stage, r_in_host, n_bytes, cudaMemcpyHostToDevice, s));
    int rc = step_device(ctx, packed_layers, stage, idx, count_dev, stride, stage, nullptr, nullptr, B, T, ws, s);
    if (rc != RM_OK) return rc;
    RM_CUDA_TRY(cudaMemcpyAsync(r_out_host, stage, n_bytes, cudaMemcpyDeviceToHost, s));
    RM_CUDA_TRY(cudaStreamSynchronize(s));
    return RM_OK;
}

int rm_device_status(rm_ctx* ctx, int* host_out, rm_stream_t stream) {
    if (!ctx || !host_out) return RM_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int v = 0;
    RM_CUDA_TRY(cudaMemcpyAsync(&v, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, s));
    RM_CUDA_TRY(cudaMemsetAsync(ctx->d_status, 0, sizeof(int), s));
    RM_CUDA_TRY(cudaStreamSynchronize(s));
    *host_out = v;
    return RM_OK;
}

int64_t rm_launch_count(const rm_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* rm_status_string(int status) {
    switch (status) {
        case RM_OK: return "ok";
        case RM_ERR_INVALID_ARG: return "invalid argument";
        case RM_ERR_SHAPE: return "shape outside the context's limits";
        case RM_ERR_ALIGN: return "pointer not 16-byte aligned";
        case RM_ERR_WORKSPACE: return "workspace missing or too small";
        case RM_ERR_CUDA: return "CUDA runtime error";
        case RM_ERR_INDEX: return "neuron index out of range or count exceeds stride";
        case RM_ERR_TIMEOUT: return "bounded device wait expired";
        case RM_ERR_UNSUPPORTED: return "not supported by this build";
        default: return "unknown status";
    }
}

}  // extern "C"
