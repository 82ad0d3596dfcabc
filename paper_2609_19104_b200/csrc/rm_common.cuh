// Shared declarations of the CUDA library: context, packed-weight geometry, launch helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rmuscle.h"

// Packed layer layout (private to the library).  Neuron n owns 3*H bf16 stored contiguously.  The chunk is cut
// into NS = 8 column slices of Hs = H/8 columns; slice j holds
//     [ Wg[n, j*Hs:(j+1)*Hs] | Wu[n, j*Hs:(j+1)*Hs] | Wd[j*Hs:(j+1)*Hs, n] ]
// so that the CTA that owns column slice j of a cluster reads one contiguous 3*Hs*2-byte piece per neuron, and a
// whole active neuron is one contiguous 6*H-byte read.
constexpr int RM_NS = 8;

struct rm_geom {
    int L, H, I, Hs;                       // Hs = H / RM_NS
    __host__ __device__ size_t neuron_elems() const { return (size_t)3 * H; }
    // element offset of (neuron n, role, column k) inside a packed layer; role 0 gate, 1 up, 2 down
    __host__ __device__ size_t off(int n, int role, int k) const {
        int j = k / Hs, kk = k - j * Hs;
        return (size_t)n * 3 * H + (size_t)j * 3 * Hs + (size_t)role * Hs + kk;
    }
};

struct rm_ctx {
    rm_model_desc desc;
    rm_geom g;
    int device;
    int sm_count;
    int* d_status;                         // device status word, then the detail word of the first error
    int status_detail;                     // detail word seen by the last rm_device_status call
    int status_log[64];                    // the whole status block of that call
    int64_t launches;                      // host-side launch counter
    // tensor-core path (rm_mlp_sm100.cu)
    int fused_clusters;                    // co-resident 8-CTA clusters of the fused layer kernel (0: unavailable)
    int fused_blocks_per_sm;               // CTAs of that kernel one SM can hold
    int path;                              // 0 auto, 1 portable kernels only, 2 fused kernel required
    int use_pdl;                           // chain layers with programmatic dependent launch
    int npc_target;                        // neurons per cluster aimed for when spreading a layer
    int count_hint;                        // expected active neurons per layer and episode (0: unknown)
    int count_hint_seen;                   // k of the last top-k / group compaction through this context (0: none yet)
    int max_clusters_override;             // > 0: cap on clusters per launch
    int l2_prefetch;                       // L2 prefetch distance (tiles) of the warp-specialised kernel
    int stream_min_tiles;                  // launches with at least this many 64-neuron tiles use the streaming variant
    int variant_override;                  // 0 auto, 1 lean kernel, 2 kernel with a dedicated staging buffer
    int last_variant;                      // kernel family of the last layer or step launched (see rm_get_info)
    // whole-step kernel (rm_mlp_persist.cu)
    int persist_clusters;                  // co-resident 8-CTA clusters of the whole-step kernel (0: unavailable)
    int persist_prefetch_kb;               // weight KB a CTA of the whole-step kernel may ask into L2 ahead of its loaders
    int persist_max_b;                     // largest batch the whole-step kernel is chosen for when the variant is automatic
    const void* persist_xbuf;              // buffer the cached tensor map below describes
    const int* persist_sync;               // the workspace's arrival counters this context has been counting on
    int persist_sync_base[16];             // their values after the launches so far
    int persist_copy_base[16];             // the same for the counters of the r_in -> r copies
    int persist_sync_dirty;                // a launch may have left them at an unknown count: clear before the next one
    alignas(64) unsigned char persist_tm[128];   // CUtensorMap of the clusters' x copies in the workspace
};

// The count the kernel selection works with: the caller's hint, else what the last compaction through this context
// was asked to keep (the counts themselves stay on the device; the host never reads them).
inline int rm_effective_count_hint(const rm_ctx* ctx) { return ctx->count_hint > 0 ? ctx->count_hint : ctx->count_hint_seen; }

extern int rm_last_cuda_error;            // cudaError_t of the last failed runtime call (diagnostics; "last_cuda_error")
#define RM_CUDA_TRY(expr)                                  \
    do {                                                   \
        cudaError_t _e = (expr);                           \
        if (_e != cudaSuccess) { rm_last_cuda_error = (int)_e; return RM_ERR_CUDA; } \
    } while (0)

// Dynamic shared-memory size a kernel has been configured for, per device: cudaFuncSetAttribute applies to the
// current device only, and one process may hold contexts on several devices.  (A race between two threads costs a
// redundant call, nothing else.)
struct rm_smem_configured {
    int bytes[64];
    bool covers(int device, int need) const { return device >= 0 && device < 64 && bytes[device] >= need; }
    void set(int device, int need) { if (device >= 0 && device < 64) bytes[device] = need; }
};

static inline bool rm_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

__device__ __forceinline__ void rm_set_status(int* status, int code) {
    if (status) atomicCAS(status, 0, code);
}
constexpr int RM_STATUS_LOG = 60;        // detail words kept per status read (the status block is 64 ints)
// The first error of a launch also leaves a detail word (where a wait gave up) next to the status word.
__device__ __forceinline__ void rm_set_status_at(int* status, int code, int detail) {
    if (!status) return;
    if (atomicCAS(status, 0, code) == 0) status[1] = detail;
    const int slot = atomicAdd(status + 2, 1);             // every error of the launch, in arrival order, while room
    if (slot < RM_STATUS_LOG) status[4 + slot] = detail;
}

__device__ __forceinline__ float rm_gelu_tanh(float g) {
    // 0.5 g (1 + tanh(sqrt(2/pi) (g + 0.044715 g^3)))
    float inner = 0.7978845608028654f * (g + 0.044715f * g * g * g);
    return 0.5f * g * (1.0f + tanhf(inner));
}

// ---- kernels implemented in the other translation units (host launchers)
int rm_launch_pack(rm_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, void* packed, float* colnorm,
                   cudaStream_t s);
int rm_launch_gather_rows(rm_ctx* ctx, const void* packed, const int32_t* idx, const int32_t* count, int64_t cap,
                          void* out, cudaStream_t s);
// Context Cache (row-sparse dense FFN on the tensor cores)
bool rm_context_supported(const rm_ctx* ctx);
size_t rm_context_workspace_bytes_impl(const rm_ctx* ctx, int r_pad);
int rm_launch_context_drift(rm_ctx* ctx, const void* x, const void* x_ref, int P, float* score, cudaStream_t s);
int rm_launch_context_ffn(rm_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, const void* x, const int32_t* rows,
                          const int32_t* count, int P, int S, int cap, const float* y_ref, float* y_out, void* ws,
                          cudaStream_t s);
int rm_launch_gather_read(rm_ctx* ctx, const void* packed, const int32_t* idx, const int32_t* count, int64_t cap,
                          cudaStream_t s);
int rm_launch_gather_read_step(rm_ctx* ctx, const void* const* packed_layers, const int32_t* idx, const int32_t* count,
                               int64_t stride, cudaStream_t s);
int rm_launch_wait_timeout(rm_ctx* ctx, unsigned polls, cudaStream_t s);
int rm_launch_mask_compact(rm_ctx* ctx, const rm_mask_src* src, int32_t* idx_out, int32_t* count_out,
                           int64_t stride, cudaStream_t s);

// Portable path (CUDA cores): any H multiple of 64, any T, any I.
struct rm_layer_args {
    const __nv_bfloat16* packed;           // packed layer
    const __nv_bfloat16* x;                // [B,T,H] bf16, or NULL when the layer normalises r_in itself
    const float* r_in;                     // [B,T,H] fp32 residual (nullable => 0 when x is given)
    float* r_out;                          // [B,T,H] fp32
    const int32_t* idx;                    // [B, idx_stride] or NULL (dense)
    const int32_t* count;                  // [B * count_stride] device counts (ignored when idx NULL)
    int64_t idx_stride;                    // elements between episodes' lists
    int64_t list_cap;                      // capacity of one list (a count above it is an error)
    int64_t count_stride;                  // elements between episodes' counts
    float* record;                         // [B, record_stride] or NULL
    int64_t record_stride;
    const float* record_scale;             // [I] or NULL
    int B, T;
    // anchor-relative update (Eq. 4); all NULL / RM_ANCHOR_NONE for the zero-fill form
    int anchor_mode;                       // RM_ANCHOR_*
    float* y_anchor;                       // [B,T,H] fp32: FFN output of the anchor step before gate and residual
    float* h_anchor;                       // [B,I,h_stride] fp32: the anchor step's hidden activations, neuron-major
    int64_t h_stride;                      // floats between neurons (>= T, multiple of 4)
    const float* gate;                     // [B,H] fp32 output gate, or NULL (= 1)
};
size_t rm_ref_workspace_bytes(const rm_ctx* ctx, int B, int T);
// Tensor-core path: H in {1024, 2048}, T <= 64 per episode, B <= 64.
int rm_fused_init(rm_ctx* ctx);
int rm_fused_debug_stamps(long long* host_out, int n);
bool rm_fused_supported(const rm_ctx* ctx, int B, int T);
int rm_launch_layer_fused(rm_ctx* ctx, const rm_layer_args& a, float* zero_buf, bool add_residual, bool pdl,
                          cudaStream_t s);
int rm_launch_layer_ref(rm_ctx* ctx, const rm_layer_args& a, void* ws, cudaStream_t s);
// Streaming tensor-core variant (whole tiles per CTA, no clusters): same shapes as the fused path.
bool rm_stream_supported(const rm_ctx* ctx, int B, int T);
int rm_stream_debug_stamps(long long* host_out);
int rm_launch_layer_stream(rm_ctx* ctx, const rm_layer_args& a, __nv_bfloat16* x_scratch, bool pdl, cudaStream_t s);
// Whole-step kernel: every layer of a step in one launch.  H in {1024, 2048}, T <= 64, B <= 16, L <= 64, zero-fill form.
struct rm_step_args {
    const void* const* packed_layers;      // host array of L device pointers
    int L;
    float* r;                              // [B,T,H] fp32: r_L on exit (r_0 on entry when r_in is NULL)
    const float* r_in;                     // [B,T,H] fp32 r_0 in another buffer (the kernel starts r as its copy), or NULL
    const int32_t* idx;                    // list (b, l) at idx + b * idx_b_stride + l * idx_l_stride; NULL: positions
    const int32_t* count;                  // count (b, l) at count[b * count_b_stride + l]; NULL: every neuron
    int64_t idx_b_stride, idx_l_stride, list_cap, count_b_stride;
    float* record;                         // record (b, l, n) at record[b * rec_b_stride + l * I + n]; NULL: none
    int64_t rec_b_stride;
    const float* record_scale;             // [L, I] or NULL
    int B, T;
    const void* x_ext;                     // [T,H] bf16: layer 0 takes this as its input instead of normalising r (L = 1 calls)
    int anchor_mode;                       // Eq. 4: RM_ANCHOR_NONE / _WRITE / _UPDATE, with the whole stack's state
    float* y_anchor;                       // [L,B,T,H]
    float* h_anchor;                       // [L,B,I,h_stride]
    int64_t h_stride;
    const float* gate;                     // [L,B,H] output gate, or NULL
};
int rm_persist_init(rm_ctx* ctx);
bool rm_persist_supported(const rm_ctx* ctx, int B, int T);
size_t rm_persist_workspace_bytes(const rm_ctx* ctx);
int rm_launch_step_persist(rm_ctx* ctx, const rm_step_args& sa, void* ws, cudaStream_t s);
int rm_persist_debug_stamps(long long* host_out, int n);
// Tiled tensor map (a 128-byte CUtensorMap, 64-byte aligned) of an fp32 residual buffer [B, T, H] with boxes of
// box_rows token rows x 128 columns of one episode, not swizzled: the target of the kernels' bulk adds.
int rm_make_out_map(void* tensor_map, const float* ptr, int B, int T, int H, int box_rows);
