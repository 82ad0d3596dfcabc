// C-ABI entry points: argument validation and dispatch.  Every step of the path runs in the library's kernels.
#include <new>
#include <cstring>
#include <cstdlib>
#include <string>

#include "rm_common.cuh"

int rm_last_cuda_error = 0;

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline bool all_aligned(std::initializer_list<const void*> ps) {
    for (const void* p : ps)
        if (p && !rm_aligned16(p)) return false;
    return true;
}

inline bool use_fused(const rm_ctx* ctx, int B, int T) {
    return ctx->path != 1 && rm_fused_supported(ctx, B, T);
}

// The whole-step kernel (variant 5).  Chosen by itself where it is measured ahead of the per-layer kernels (single
// episodes; us per step, cold L2: lean per-layer kernel / streaming kernel / whole-step kernel):
//   H = 2048, I = 16384:  K =  492: 236 / 572 / 262    820: 265 / 571 / 262    1147: 360 / 571 / 266
//                         1639: 377 / 577 / 273    3277: 605 / 577 / 308    4916: 829 / 554 / 462
//                         6882: 1058 / 584 / 532    7373: 1066 / 605 / 544    8192: 1183 / 624 / 652
//                         9012: 1279 / 665 / 687    9503: 1301 / 1039 / 701    12288: 1632 / 1139 / 871
//                         14746: 1962 / 1114 / 960    16384 (every neuron listed): 2158 / 1130 / 1081
//   H = 1024, I = 4096:   K =  820: 176 / 344 / 188    902: 178 / 345 / 190    984: 200 / 343 / 193
//                         1024: 199 / 345 / 193    1229: 231 / 345 / 195    2048: 270 / 346 / 203    4096: 404 / 337 / 291
// The streaming kernel's time steps up with every wave of 64-neuron tiles over the SMs (148 tiles per wave), the lean
// kernel's with every 64-neuron tile beyond 15; the whole-step kernel grows evenly with K and has a fixed cost of
// ~10-15 us per layer.  So, with K the caller's count hint (the whole layer for a dense pass): at H = 1024 from 23.5 %
// of the neurons upwards; at H = 2048 from 5 % upwards, except where the streaming kernel's single wave is nearly full
// (47 % of the neurons up to 148 tiles).  Without a hint at H = 2048 it is chosen as well (it adapts to the counts on
// the device), at H = 1024 the lean kernel.  Batches stay with the streaming kernel.  `steps`: a whole stack (false:
// the one-layer entry, which would pay the kernel's set-up for a single layer).
inline bool use_persist(const rm_ctx* ctx, int B, int T, bool masked, bool steps) {
    if (ctx->path == 1 || !rm_persist_supported(ctx, B, T)) return false;
    if (ctx->variant_override == 5) return true;
    if (ctx->variant_override != 0 || B > ctx->persist_max_b || !steps) return false;
    const long long I = ctx->g.I, K = masked ? rm_effective_count_hint(ctx) : I;
    if (ctx->g.H == 2048) {
        if (K <= 0) return true;
        if (K * 100 < I * 5) return false;
        return !(K * 100 > I * 47 && (K + 63) / 64 <= ctx->sm_count);
    }
    return K > 0 && K * 1000 >= I * 235;
}

inline void* persist_ws(const rm_ctx* ctx, void* ws, int B, int T) {
    const size_t r_bytes = align_up((size_t)B * T * ctx->g.H * sizeof(float), 256);
    return static_cast<char*>(ws) + 4 * r_bytes + align_up(rm_ref_workspace_bytes(ctx, B, T), 256);
}

// The streaming variant (whole tiles per CTA) pays off only when a launch has about one 64-neuron tile per SM (one SM
// gathers at most ~38 GB/s with 16-byte cp.async and adds at most ~20 GB/s with red.global, so a tile costs it
// ~25 us); below that the cluster kernels, which spread a tile over 8 SMs, win.  H = 1024 only: at H = 2048 the
// warp-specialised cluster kernel is ahead at every size measured.  `masked` says whether a count is in play.
// anchor_write: the anchor step of Eq. 4 adds two boxes per block (y_anchor and the output) and stores h_anchor; measured
// on the anchor schedule it stays behind the cluster kernels at 64 tiles (352 against 334 us per step), so it keeps
// the threshold of about a tile per SM
inline bool use_stream(const rm_ctx* ctx, bool masked, int B, int T, bool anchor_write = false) {
    if (ctx->path == 1 || !rm_stream_supported(ctx, B, T)) return false;
    if (ctx->variant_override == 4) return true;
    if (ctx->variant_override != 0 && ctx->variant_override != 5) return false;   // 5: a call the whole-step kernel does not cover
    const int per_episode = masked ? rm_effective_count_hint(ctx) : ctx->g.I;
    if (per_episode <= 0) return false;
    const long long tiles = (long long)((per_episode + 63) / 64) * B;
    return tiles >= (anchor_write && ctx->stream_min_tiles < 112 ? 112 : ctx->stream_min_tiles);
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
    c->status_detail = 0;
    // measured crossover with the cluster kernels.  H = 1024: at 32 tiles the lean kernel is far ahead (270 against
    // 370 us per step); at 48 the two are level on 3 episodes x 16 tiles (127 against 126) and the streaming variant
    // is 7 % ahead on one episode of 48 tiles (378 against 350); at 64 it is 10 % ahead, at 80 by 30 %.
    // H = 2048: the warp-specialised kernel is ahead at 52 tiles (512 against 582), level at 64, behind at 96 (50
    // against 38 us per layer).
    c->stream_min_tiles = desc->H == 2048 ? 64 : 48;
    c->d_status = nullptr;
    cudaDeviceProp prop;
    if (cudaGetDevice(&c->device) != cudaSuccess || cudaGetDeviceProperties(&prop, c->device) != cudaSuccess ||
        cudaMalloc(&c->d_status, 256) != cudaSuccess || cudaMemset(c->d_status, 0, 256) != cudaSuccess) {
        if (c->d_status) cudaFree(c->d_status);
        delete c;
        return RM_ERR_CUDA;
    }
    c->sm_count = prop.multiProcessorCount;
    c->path = 0;
    c->use_pdl = 1;
    c->npc_target = 64;
    c->count_hint = 0;
    c->count_hint_seen = 0;
    c->max_clusters_override = 0;
    c->variant_override = 0;
    c->l2_prefetch = 0;
    c->fused_clusters = 0;
    c->fused_blocks_per_sm = 0;
    c->last_variant = 0;
    c->persist_clusters = 0;
    c->persist_max_b = 1;
    c->persist_prefetch_kb = 0;
    c->persist_xbuf = nullptr;
    c->persist_sync = nullptr;
    c->persist_sync_dirty = 0;
    for (int b = 0; b < 16; ++b) c->persist_sync_base[b] = c->persist_copy_base[b] = 0;
    if (prop.major == 10) { rm_fused_init(c); rm_persist_init(c); }   // failure leaves the portable path in charge
    cudaGetLastError();
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
    // three rotating residual-stream buffers, the host variant's staging buffer, then the portable path's scratch
    size_t r_bytes = align_up((size_t)B * T * ctx->g.H * sizeof(float), 256);
    return 4 * r_bytes + align_up(rm_ref_workspace_bytes(ctx, B, T), 256) + rm_persist_workspace_bytes(ctx);
}

int rm_pack_weights(rm_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, void* packed_out,
                    float* down_colnorm, rm_stream_t stream) {
    if (!ctx || !Wg || !Wu || !Wd || !packed_out) return RM_ERR_INVALID_ARG;
    if (!all_aligned({Wg, Wu, Wd, packed_out, down_colnorm})) return RM_ERR_ALIGN;
    return rm_launch_pack(ctx, Wg, Wu, Wd, packed_out, down_colnorm, static_cast<cudaStream_t>(stream));
}

int rm_debug_gather_read(rm_ctx* ctx, const void* packed_layer, const int32_t* idx, const int32_t* count_dev,
                         int64_t list_cap, rm_stream_t stream) {
    if (!ctx || !packed_layer || (idx && !count_dev) || list_cap < 0) return RM_ERR_INVALID_ARG;
    if (!all_aligned({packed_layer, idx})) return RM_ERR_ALIGN;
    return rm_launch_gather_read(ctx, packed_layer, idx, count_dev, idx ? list_cap : ctx->g.I,
                                 static_cast<cudaStream_t>(stream));
}

int rm_debug_gather_read_step(rm_ctx* ctx, const void* const* packed_layers, const int32_t* idx, const int32_t* count_dev,
                              int64_t stride, rm_stream_t stream) {
    if (!ctx || !packed_layers || (idx && (!count_dev || stride < 1))) return RM_ERR_INVALID_ARG;
    for (int l = 0; l < ctx->g.L; ++l) {
        if (!packed_layers[l]) return RM_ERR_INVALID_ARG;
        if (!rm_aligned16(packed_layers[l])) return RM_ERR_ALIGN;
    }
    if (!all_aligned({idx})) return RM_ERR_ALIGN;
    return rm_launch_gather_read_step(ctx, packed_layers, idx, count_dev, stride, static_cast<cudaStream_t>(stream));
}

int rm_debug_wait_timeout(rm_ctx* ctx, int polls, rm_stream_t stream) {
    if (!ctx || polls < 1 || polls > (1 << 20)) return RM_ERR_INVALID_ARG;
    return rm_launch_wait_timeout(ctx, (unsigned)polls, static_cast<cudaStream_t>(stream));
}

int rm_gather_weights(rm_ctx* ctx, const void* packed_layer, const int32_t* idx, const int32_t* count_dev,
                      int64_t list_cap, void* compact_out, rm_stream_t stream) {
    if (!ctx || !packed_layer || !idx || !count_dev || !compact_out || list_cap < 0) return RM_ERR_INVALID_ARG;
    if (!all_aligned({packed_layer, idx, compact_out})) return RM_ERR_ALIGN;
    if (compact_out == packed_layer) return RM_ERR_INVALID_ARG;
    return rm_launch_gather_rows(ctx, packed_layer, idx, count_dev, list_cap, compact_out,
                                 static_cast<cudaStream_t>(stream));
}

static int context_pad(int R_max) { return R_max <= 64 ? 64 : (R_max <= 128 ? 128 : 256); }

int rm_context_drift(rm_ctx* ctx, const void* x, const void* x_ref, int P, float* score_out, rm_stream_t stream) {
    if (!ctx || !x || !x_ref || !score_out || P < 0) return RM_ERR_INVALID_ARG;
    if (ctx->g.H % 8 != 0) return RM_ERR_UNSUPPORTED;
    if (!all_aligned({x, x_ref, score_out})) return RM_ERR_ALIGN;
    if (P == 0) return RM_OK;
    return rm_launch_context_drift(ctx, x, x_ref, P, score_out, static_cast<cudaStream_t>(stream));
}

constexpr int RM_CONTEXT_MAX_ROWS = 1024;      // four passes of 256 rows over the weights

size_t rm_context_workspace_bytes(const rm_ctx* ctx, int R_max) {
    if (!ctx || R_max < 1 || R_max > RM_CONTEXT_MAX_ROWS || !rm_context_supported(ctx)) return 0;
    return rm_context_workspace_bytes_impl(ctx, context_pad(R_max));
}

int rm_context_ffn(rm_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, const void* x, const int32_t* rows,
                   const int32_t* count_dev, int P, int S, int R_max, const float* y_ref, float* y_out, void* ws,
                   size_t ws_bytes, rm_stream_t stream) {
    if (!ctx || !Wg || !Wu || !Wd || !x || !rows || !count_dev || !y_ref || !y_out || P < 0 || S < 0) return RM_ERR_INVALID_ARG;
    if (!rm_context_supported(ctx)) return RM_ERR_UNSUPPORTED;
    if (R_max < 1 || R_max > RM_CONTEXT_MAX_ROWS || S > R_max) return RM_ERR_SHAPE;
    if (!all_aligned({Wg, Wu, Wd, x, rows, y_ref, y_out, ws})) return RM_ERR_ALIGN;
    if (!ws || ws_bytes < rm_context_workspace_bytes(ctx, R_max)) return RM_ERR_WORKSPACE;
    // rows beyond 256 take further passes; a single pass rounds its capacity up to the tile it runs in
    return rm_launch_context_ffn(ctx, Wg, Wu, Wd, x, rows, count_dev, P, S, R_max <= 256 ? context_pad(R_max) : R_max, y_ref,
                                 y_out, ws, static_cast<cudaStream_t>(stream));
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
    if ((src->reduce == RM_REDUCE_TOPK || src->reduce == RM_REDUCE_GROUP) && src->I == ctx->g.I)
        ctx->count_hint_seen = src->k < src->I ? src->k : src->I;
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
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t r_bytes = align_up((size_t)T * ctx->g.H * sizeof(float), 256);
    if (use_fused(ctx, 1, T)) {
        // y accumulates the CTAs' partial sums with atomics: start it from the residual (or zero)
        if (y != residual) {
            if (residual) RM_CUDA_TRY(cudaMemcpyAsync(y, residual, (size_t)T * ctx->g.H * sizeof(float),
                                                      cudaMemcpyDeviceToDevice, s));
            else RM_CUDA_TRY(cudaMemsetAsync(y, 0, (size_t)T * ctx->g.H * sizeof(float), s));
        }
        if (use_persist(ctx, 1, T, count_dev != nullptr, false)) {
            // the whole-step kernel on a stack of one layer whose input is the caller's x
            const void* one[1] = {packed_layer};
            rm_step_args sa{};
            sa.packed_layers = one;
            sa.L = 1;
            sa.r = y;
            sa.idx = idx;
            sa.count = count_dev;
            sa.idx_b_stride = 0;
            sa.idx_l_stride = 0;
            sa.list_cap = ctx->g.I;
            sa.count_b_stride = 0;
            sa.record = record_out;
            sa.rec_b_stride = 0;
            sa.record_scale = record_scale;
            sa.B = 1;
            sa.T = T;
            sa.x_ext = x;
            ctx->last_variant = 5;
            return rm_launch_step_persist(ctx, sa, persist_ws(ctx, ws, 1, T), s);
        }
        if (use_stream(ctx, count_dev != nullptr, 1, T)) {
            ctx->last_variant = 4;
            return rm_launch_layer_stream(ctx, a, nullptr, false, s);
        }
        return rm_launch_layer_fused(ctx, a, nullptr, false, false, s);
    }
    if (ctx->path == 2) return RM_ERR_UNSUPPORTED;
    ctx->last_variant = 0;
    return rm_launch_layer_ref(ctx, a, static_cast<char*>(ws) + 4 * r_bytes, s);
}

namespace {
struct AnchorIO {                      // whole-stack anchor state (Eq. 4); mode RM_ANCHOR_NONE and NULLs for none
    int mode = RM_ANCHOR_NONE;
    float* y = nullptr;                // [L,B,T,H]
    float* h = nullptr;                // [L,B,I,h_stride]
    int64_t h_stride = 0;
    const float* gate = nullptr;       // [L,B,H]
};
}  // namespace

static int step_device(rm_ctx* ctx, const void* const* packed_layers, const float* r_in, const int32_t* idx,
                       const int32_t* count_dev, int64_t stride, float* r_out, float* records_out,
                       const float* record_scale, int B, int T, void* ws, cudaStream_t s,
                       const AnchorIO& an = AnchorIO()) {
    const rm_geom& g = ctx->g;
    const size_t n_bytes = (size_t)B * T * g.H * sizeof(float);
    const size_t r_bytes = align_up(n_bytes, 256);
    char* layer_ws = static_cast<char*>(ws) + 4 * r_bytes;
    if (use_persist(ctx, B, T, count_dev != nullptr, true)) {
        // the whole step in one launch: the layers add into r_out in place (the kernel starts it as a copy of r_in)
        rm_step_args sa{};
        sa.packed_layers = packed_layers;
        sa.L = g.L;
        sa.r = r_out;
        sa.r_in = r_out != r_in ? r_in : nullptr;
        sa.idx = idx;
        sa.count = count_dev;
        sa.idx_b_stride = (int64_t)g.L * stride;
        sa.idx_l_stride = stride;
        sa.list_cap = idx ? stride : g.I;
        sa.count_b_stride = g.L;
        sa.record = records_out;
        sa.rec_b_stride = (int64_t)g.L * g.I;
        sa.record_scale = record_scale;
        sa.B = B;
        sa.T = T;
        sa.anchor_mode = an.mode;
        sa.y_anchor = an.y;
        sa.h_anchor = an.h;
        sa.h_stride = an.h_stride;
        sa.gate = an.gate;
        ctx->last_variant = 5;
        return rm_launch_step_persist(ctx, sa, persist_ws(ctx, ws, B, T), s);
    }
    const bool fused = use_fused(ctx, B, T);
    if (!fused && ctx->path == 2) return RM_ERR_UNSUPPORTED;
    float* rot[3] = {reinterpret_cast<float*>(static_cast<char*>(ws)),
                     reinterpret_cast<float*>(static_cast<char*>(ws) + r_bytes),
                     reinterpret_cast<float*>(static_cast<char*>(ws) + 2 * r_bytes)};
    // Fused path: layer l reads rot[l%3] (the caller's r_in for l = 0), accumulates into rot[(l+1)%3] and clears
    // rot[(l+2)%3] for the layer after next; the last layer accumulates straight into r_out when that is a
    // different buffer from r_in.
    const bool stream = fused && use_stream(ctx, count_dev != nullptr, B, T, an.mode == RM_ANCHOR_WRITE);
    const bool direct_out = fused && r_out != r_in;
    if (fused && !stream) {
        RM_CUDA_TRY(cudaMemsetAsync(g.L == 1 && direct_out ? r_out : rot[1], 0, n_bytes, s));
        if (direct_out && g.L > 1) RM_CUDA_TRY(cudaMemsetAsync(r_out, 0, n_bytes, s));
    }
    // the anchor step's outputs are accumulated by the CTAs' atomics: start them from zero
    if (fused && an.mode == RM_ANCHOR_WRITE)
        RM_CUDA_TRY(cudaMemsetAsync(an.y, 0, (size_t)g.L * n_bytes, s));
    const float* cur = r_in;
    for (int l = 0; l < g.L; ++l) {
        rm_layer_args a{};
        a.packed = static_cast<const __nv_bfloat16*>(packed_layers[l]);
        a.x = nullptr;
        a.r_in = cur;
        a.idx = idx ? idx + (size_t)l * stride : nullptr;
        a.count = count_dev ? count_dev + l : nullptr;
        a.idx_stride = (int64_t)g.L * stride;
        a.list_cap = idx ? stride : g.I;
        a.count_stride = g.L;
        a.record = records_out ? records_out + (size_t)l * g.I : nullptr;
        a.record_stride = (int64_t)g.L * g.I;
        a.record_scale = record_scale ? record_scale + (size_t)l * g.I : nullptr;
        a.B = B;
        a.T = T;
        a.anchor_mode = an.mode;
        a.y_anchor = an.y ? an.y + (size_t)l * B * T * g.H : nullptr;
        a.h_anchor = an.h ? an.h + (size_t)l * B * g.I * an.h_stride : nullptr;
        a.h_stride = an.h_stride;
        a.gate = an.gate ? an.gate + (size_t)l * B * g.H : nullptr;
        int rc;
        if (stream) {
            // two buffers in turn: the preparation kernel writes the residual part of the output, the tiles add theirs
            const bool last = l == g.L - 1;
            a.r_out = (last && direct_out) ? r_out : rot[l & 1];
            ctx->last_variant = 4;
            rc = rm_launch_layer_stream(ctx, a, reinterpret_cast<__nv_bfloat16*>(layer_ws), ctx->use_pdl && l > 0, s);
            cur = a.r_out;
        } else if (fused) {
            const bool last = l == g.L - 1;
            a.r_out = (last && direct_out) ? r_out : rot[(l + 1) % 3];
            // the buffer cleared here is the output of layer l+1 (unless that layer writes to r_out directly); it
            // was the input of layer l-1, which has completed by the time this layer passes its dependency wait
            float* zero = (l + 1 < g.L && !(l + 1 == g.L - 1 && direct_out)) ? rot[(l + 2) % 3] : nullptr;
            rc = rm_launch_layer_fused(ctx, a, zero, true, ctx->use_pdl && l > 0, s);
            cur = a.r_out;
        } else {
            a.r_out = r_out;                               // in place after the first layer
            ctx->last_variant = 0;
            rc = rm_launch_layer_ref(ctx, a, layer_ws, s);
            cur = r_out;
        }
        if (rc != RM_OK) return rc;
    }
    if (fused && !direct_out) RM_CUDA_TRY(cudaMemcpyAsync(r_out, cur, n_bytes, cudaMemcpyDeviceToDevice, s));
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

int rm_action_expert_step_ex(rm_ctx* ctx, const void* const* packed_layers, const float* r_in, const int32_t* idx,
                             const int32_t* count_dev, int64_t stride, float* r_out, float* records_out,
                             const float* record_scale, int B, int T, int anchor_mode, float* y_anchor,
                             float* h_anchor, int64_t h_stride, const float* out_gate, void* ws, size_t ws_bytes,
                             rm_stream_t stream) {
    if (!ctx || !packed_layers || !r_in || !r_out || B < 0 || T < 0) return RM_ERR_INVALID_ARG;
    if (idx && (!count_dev || stride < 1)) return RM_ERR_INVALID_ARG;
    if (idx && records_out) return RM_ERR_INVALID_ARG;
    if (anchor_mode != RM_ANCHOR_NONE && anchor_mode != RM_ANCHOR_WRITE && anchor_mode != RM_ANCHOR_UPDATE)
        return RM_ERR_INVALID_ARG;
    if (anchor_mode != RM_ANCHOR_NONE) {
        if (!y_anchor || !h_anchor || h_stride < T) return RM_ERR_INVALID_ARG;
        if (h_stride % 4 != 0) return RM_ERR_ALIGN;
        // the anchor state is read (or accumulated) while the outputs are written: no overlap with them
        if (y_anchor == r_out || y_anchor == r_in) return RM_ERR_INVALID_ARG;
    }
    if (B > ctx->desc.B_max || T > ctx->desc.T_max) return RM_ERR_SHAPE;
    for (int l = 0; l < ctx->g.L; ++l) {
        if (!packed_layers[l]) return RM_ERR_INVALID_ARG;
        if (!rm_aligned16(packed_layers[l])) return RM_ERR_ALIGN;
    }
    if (!all_aligned({r_in, idx, r_out, records_out, record_scale, ws, y_anchor, h_anchor, out_gate}))
        return RM_ERR_ALIGN;
    if (idx && (stride % 4) != 0) return RM_ERR_ALIGN;
    if (B == 0 || T == 0) return RM_OK;
    if (!ws || ws_bytes < rm_workspace_bytes(ctx, B, T)) return RM_ERR_WORKSPACE;
    AnchorIO an;
    an.mode = anchor_mode;
    if (anchor_mode != RM_ANCHOR_NONE) { an.y = y_anchor; an.h = h_anchor; an.h_stride = h_stride; }
    an.gate = out_gate;
    return step_device(ctx, packed_layers, r_in, idx, count_dev, stride, r_out, records_out, record_scale, B, T, ws,
                       static_cast<cudaStream_t>(stream), an);
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
    // the fourth residual-stream buffer of the workspace is the staging copy
    float* stage = reinterpret_cast<float*>(static_cast<char*>(ws) + 3 * align_up(n_bytes, 256));
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
    int v[64] = {0};
    RM_CUDA_TRY(cudaMemcpyAsync(v, ctx->d_status, sizeof(v), cudaMemcpyDeviceToHost, s));
    RM_CUDA_TRY(cudaMemsetAsync(ctx->d_status, 0, sizeof(v), s));
    RM_CUDA_TRY(cudaStreamSynchronize(s));
    *host_out = v[0];
    if (v[0] != 0) ctx->persist_sync_dirty = 1;                 // a whole-step launch may have stopped half way
    ctx->status_detail = v[0] ? v[1] : 0;
    std::memcpy(ctx->status_log, v, sizeof(v));
    return RM_OK;
}

int64_t rm_launch_count(const rm_ctx* ctx) { return ctx ? ctx->launches : 0; }

int rm_set_option(rm_ctx* ctx, const char* name, int value) {
    if (!ctx || !name) return RM_ERR_INVALID_ARG;
    const std::string n(name);
    if (n == "path") {
        if (value < 0 || value > 2) return RM_ERR_INVALID_ARG;
        ctx->path = value;
    } else if (n == "pdl") {
        ctx->use_pdl = value != 0;
    } else if (n == "neurons_per_cluster") {
        if (value < 1) return RM_ERR_INVALID_ARG;
        ctx->npc_target = value;
    } else if (n == "count_hint") {
        if (value < 0) return RM_ERR_INVALID_ARG;
        ctx->count_hint = value;
    } else if (n == "variant") {
        if (value < 0 || value > 5) return RM_ERR_INVALID_ARG;
        ctx->variant_override = value;
    } else if (n == "persist_prefetch_kb") {
        if (value < 0 || value > 4096) return RM_ERR_INVALID_ARG;
        ctx->persist_prefetch_kb = value;
    } else if (n == "persist_max_batch") {
        if (value < 0 || value > 16) return RM_ERR_INVALID_ARG;
        ctx->persist_max_b = value;
    } else if (n == "stream_min_tiles") {
        if (value < 1) return RM_ERR_INVALID_ARG;
        ctx->stream_min_tiles = value;
    } else if (n == "l2_prefetch") {
        if (value < 0 || value > 16) return RM_ERR_INVALID_ARG;
        ctx->l2_prefetch = value;
    } else if (n == "max_clusters") {
        if (value < 0) return RM_ERR_INVALID_ARG;
        ctx->max_clusters_override = value;
    } else {
        return RM_ERR_INVALID_ARG;
    }
    return RM_OK;
}

int rm_get_info(const rm_ctx* ctx, const char* name, int* out) {
    if (!name || !out) return RM_ERR_INVALID_ARG;
    const std::string n(name);
    if (n == "last_cuda_error") { *out = rm_last_cuda_error; return RM_OK; }   // process-wide: needs no context
    if (!ctx) return RM_ERR_INVALID_ARG;
    if (n == "fused_clusters") *out = ctx->fused_clusters;
    else if (n == "fused_blocks_per_sm") *out = ctx->fused_blocks_per_sm;
    else if (n == "sm_count") *out = ctx->sm_count;
    else if (n == "persist_clusters") *out = ctx->persist_clusters;
    else if (n == "last_variant") *out = ctx->last_variant;
    else if (n == "path") *out = ctx->path;
    else if (n == "status_detail") *out = ctx->status_detail;
    else if (n == "status_log_count") *out = ctx->status_log[2] < RM_STATUS_LOG ? ctx->status_log[2] : RM_STATUS_LOG;
    else if (n.rfind("status_log:", 0) == 0) {
        const int i = std::atoi(n.c_str() + 11);
        if (i < 0 || i >= RM_STATUS_LOG) return RM_ERR_INVALID_ARG;
        *out = ctx->status_log[4 + i];
    }
    else return RM_ERR_INVALID_ARG;
    return RM_OK;
}

int rm_debug_phase_times(rm_ctx* ctx, long long* host_out, int n) {
    if (!ctx || !host_out) return RM_ERR_INVALID_ARG;
    if (n == -64) return rm_stream_debug_stamps(host_out);      // the streaming kernel's stamps (first tile of CTA 0)
    if (n <= -(1 << 20)) return rm_persist_debug_stamps(host_out, -n - (1 << 20));   // the whole-step kernel's stamps
    return rm_fused_debug_stamps(host_out, n);
}

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
