// Portable CUDA-core path of the masked gated MLP: three plain kernels per layer (RMSNorm -> bf16 x, gate/up
// dot products + GeLU-tanh GLU into a compact fp32 h, down projection + residual).  It accepts any H that is a
// multiple of 64, any T and any I; the tensor-core path covers the shapes that matter for speed and this one
// covers everything else.
#include <mutex>

#include "rm_common.cuh"

namespace {

constexpr int GU_WARPS = 8;        // neurons per CTA in the gate/up kernel (one warp each)
constexpr int DN_THREADS = 128;    // two output columns per thread
constexpr int DN_TOK = 8;          // tokens per CTA in the down kernel
constexpr int DN_CHUNK = 64;       // neurons staged per iteration

__device__ __forceinline__ int clamp_count(const rm_layer_args& a, int b, const rm_geom& g, int* status) {
    if (!a.count) return g.I;          // a count without a list: the leading `count` neurons (compact layer)
    int c = a.count[(size_t)b * a.count_stride];
    int cap = (int)(a.list_cap < (int64_t)g.I ? a.list_cap : (int64_t)g.I);
    if (c < 0 || c > cap) {
        rm_set_status(status, RM_ERR_INDEX);
        c = c < 0 ? 0 : cap;
    }
    return c;
}

// x[b,t,:] = bf16( r[b,t,:] / sqrt(mean r^2 + 1e-6) ), one CTA per token row
__global__ void __launch_bounds__(256) ref_norm_kernel(const float* __restrict__ r, __nv_bfloat16* __restrict__ x,
                                                       int H) {
    __shared__ float part[8];
    const float* row = r + (size_t)blockIdx.x * H;
    float ss = 0.0f;
    for (int k = threadIdx.x; k < H; k += blockDim.x) ss = fmaf(row[k], row[k], ss);
    for (int d = 16; d > 0; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.0f;
    for (int w = 0; w < 8; ++w) tot += part[w];
    const float inv = 1.0f / sqrtf(tot / (float)H + 1e-6f);
    for (int k = threadIdx.x; k < H; k += blockDim.x)
        x[(size_t)blockIdx.x * H + k] = __float2bfloat16_rn(row[k] * inv);
}

__device__ __forceinline__ void fma8(const uint4& a, const uint4& b, float& acc) {
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 fa = __bfloat1622float2(pa[i]), fb = __bfloat1622float2(pb[i]);
        acc = fmaf(fa.x, fb.x, acc);
        acc = fmaf(fa.y, fb.y, acc);
    }
}

// h[b,t,j] = gelu_tanh(<x_t, Wg_n>) * <x_t, Wu_n>, n = idx[j]; one warp per neuron, lanes split the H columns.
__global__ void __launch_bounds__(GU_WARPS * 32) ref_gateup_kernel(rm_layer_args a, rm_geom g,
                                                                   const __nv_bfloat16* __restrict__ x,
                                                                   float* __restrict__ h, int* status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.y;
    const int cnt = clamp_count(a, b, g, status);
    const int j = blockIdx.x * GU_WARPS + warp;
    if (j >= cnt) return;
    int n = a.idx ? a.idx[(size_t)b * a.idx_stride + j] : j;
    bool bad = n < 0 || n >= g.I;
    if (bad) { rm_set_status(status, RM_ERR_INDEX); n = 0; }

    // stage this neuron's gate and up rows (natural column order) in shared memory
    uint4* wg = reinterpret_cast<uint4*>(smem_raw) + (size_t)warp * (2 * g.H / 8);
    uint4* wu = wg + g.H / 8;
    const int hs8 = g.Hs / 8;
    for (int k8 = lane; k8 < g.H / 8; k8 += 32) {
        int jslice = k8 / hs8, kk8 = k8 - jslice * hs8;
        const uint4* src = reinterpret_cast<const uint4*>(a.packed + (size_t)n * 3 * g.H + (size_t)jslice * 3 * g.Hs);
        wg[k8] = src[kk8];
        wu[k8] = src[hs8 + kk8];
    }
    __syncwarp();

    float rec = 0.0f;
    for (int t = 0; t < a.T; ++t) {
        const uint4* xr = reinterpret_cast<const uint4*>(x + ((size_t)b * a.T + t) * g.H);
        float ag = 0.0f, au = 0.0f;
        for (int k8 = lane; k8 < g.H / 8; k8 += 32) {
            uint4 xv = xr[k8];
            fma8(xv, wg[k8], ag);
            fma8(xv, wu[k8], au);
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            ag += __shfl_xor_sync(0xffffffffu, ag, d);
            au += __shfl_xor_sync(0xffffffffu, au, d);
        }
        float hv = bad ? 0.0f : rm_gelu_tanh(ag) * au;
        rec += fabsf(hv);
        if (lane == 0) {
            // Eq. 4: the anchor step retains h, a later step contributes its difference from the anchor's h
            if (a.anchor_mode != RM_ANCHOR_NONE && !bad) {
                float* ha = a.h_anchor + ((size_t)b * g.I + n) * a.h_stride + t;
                if (a.anchor_mode == RM_ANCHOR_WRITE) *ha = hv;
                else hv -= *ha;
            }
            h[((size_t)b * a.T + t) * g.I + j] = hv;
        }
    }
    if (a.record && lane == 0 && !bad)
        a.record[(size_t)b * a.record_stride + n] = a.record_scale ? rec * a.record_scale[n] : rec;
}

// y[b,t,c] = r[b,t,c] + sum_j h[b,t,j] * Wd[c, idx[j]]
__global__ void __launch_bounds__(DN_THREADS) ref_down_kernel(rm_layer_args a, rm_geom g, const float* __restrict__ h,
                                                              int* status) {
    __shared__ float sh_h[DN_TOK][DN_CHUNK];
    __shared__ int sh_n[DN_CHUNK];
    const int b = blockIdx.z;
    const int t0 = blockIdx.y * DN_TOK;
    const int c = (blockIdx.x * DN_THREADS + threadIdx.x) * 2;
    const bool col_ok = c < g.H;
    const int cnt = clamp_count(a, b, g, status);
    float acc[DN_TOK][2];
#pragma unroll
    for (int i = 0; i < DN_TOK; ++i) acc[i][0] = acc[i][1] = 0.0f;
    const int jslice = col_ok ? c / g.Hs : 0;
    const size_t col_off = (size_t)jslice * 3 * g.Hs + 2 * g.Hs + (c - jslice * g.Hs);

    for (int j0 = 0; j0 < cnt; j0 += DN_CHUNK) {
        const int m = min(DN_CHUNK, cnt - j0);
        __syncthreads();
        for (int e = threadIdx.x; e < DN_CHUNK; e += DN_THREADS) {
            int n = 0;
            if (e < m) {
                n = a.idx ? a.idx[(size_t)b * a.idx_stride + j0 + e] : j0 + e;
                if (n < 0 || n >= g.I) n = -1;       // already reported by the gate/up kernel; contributes 0
            }
            sh_n[e] = n;
        }
        for (int e = threadIdx.x; e < DN_TOK * DN_CHUNK; e += DN_THREADS) {
            int tt = e / DN_CHUNK, q = e - tt * DN_CHUNK;
            int t = t0 + tt;
            sh_h[tt][q] = (t < a.T && q < m) ? h[((size_t)b * a.T + t) * g.I + j0 + q] : 0.0f;
        }
        __syncthreads();
        if (col_ok) {
            for (int q = 0; q < m; ++q) {
                int n = sh_n[q];
                if (n < 0) continue;
                float2 w = __bfloat1622float2(
                    *reinterpret_cast<const __nv_bfloat162*>(a.packed + (size_t)n * 3 * g.H + col_off));
#pragma unroll
                for (int tt = 0; tt < DN_TOK; ++tt) {
                    acc[tt][0] = fmaf(sh_h[tt][q], w.x, acc[tt][0]);
                    acc[tt][1] = fmaf(sh_h[tt][q], w.y, acc[tt][1]);
                }
            }
        }
    }
    if (!col_ok) return;
#pragma unroll
    for (int tt = 0; tt < DN_TOK; ++tt) {
        int t = t0 + tt;
        if (t >= a.T) break;
        size_t o = ((size_t)b * a.T + t) * g.H + c;
        float2 base = a.r_in ? *reinterpret_cast<const float2*>(a.r_in + o) : make_float2(0.0f, 0.0f);
        float2 y = make_float2(acc[tt][0], acc[tt][1]);
        if (a.anchor_mode == RM_ANCHOR_WRITE) {
            *reinterpret_cast<float2*>(a.y_anchor + o) = y;
        } else if (a.anchor_mode == RM_ANCHOR_UPDATE) {
            const float2 ya = *reinterpret_cast<const float2*>(a.y_anchor + o);
            y.x += ya.x;
            y.y += ya.y;
        }
        const float2 gt = a.gate ? *reinterpret_cast<const float2*>(a.gate + (size_t)b * g.H + c) : make_float2(1.0f, 1.0f);
        *reinterpret_cast<float2*>(a.r_out + o) = make_float2(base.x + gt.x * y.x, base.y + gt.y * y.y);
    }
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

size_t rm_ref_workspace_bytes(const rm_ctx* ctx, int B, int T) {
    size_t x_bytes = align_up((size_t)B * T * ctx->g.H * sizeof(__nv_bfloat16), 256);
    size_t h_bytes = align_up((size_t)B * T * ctx->g.I * sizeof(float), 256);
    return x_bytes + h_bytes;
}

namespace {
// The gate/up kernel's dynamic shared-memory limit, per device: only ever raised, so that two users of the kernel
// with different H (a context's portable path and the allocation-free entry point) cannot lower it under each other.
constexpr int RM_MAX_DEVICES = 64;
std::mutex g_gateup_mutex;
int g_gateup_smem[RM_MAX_DEVICES] = {};
constexpr size_t RM_GATEUP_SMEM_LIMIT = 227 * 1024;               // opt-in shared memory of one CTA on sm_100

int ensure_gateup_smem(size_t smem) {
    if (smem <= 48 * 1024) return RM_OK;
    if (smem > RM_GATEUP_SMEM_LIMIT) return RM_ERR_SHAPE;
    int dev = -1;
    RM_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= RM_MAX_DEVICES) return RM_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_gateup_mutex);
    if (g_gateup_smem[dev] < (int)smem) {
        RM_CUDA_TRY(cudaFuncSetAttribute(ref_gateup_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        g_gateup_smem[dev] = (int)smem;
    }
    return RM_OK;
}
}  // namespace

int rm_launch_layer_ref(rm_ctx* ctx, const rm_layer_args& a, void* ws, cudaStream_t s) {
    const rm_geom& g = ctx->g;
    if (a.B <= 0 || a.T <= 0) return RM_OK;
    size_t x_bytes = align_up((size_t)a.B * a.T * g.H * sizeof(__nv_bfloat16), 256);
    __nv_bfloat16* xbuf = static_cast<__nv_bfloat16*>(ws);
    float* h = reinterpret_cast<float*>(static_cast<char*>(ws) + x_bytes);
    const __nv_bfloat16* x = a.x;
    if (!x) {
        ref_norm_kernel<<<a.B * a.T, 256, 0, s>>>(a.r_in, xbuf, g.H);
        ctx->launches++;
        x = xbuf;
    }
    size_t smem = (size_t)GU_WARPS * 2 * g.H * sizeof(__nv_bfloat16);
    {
        const int rc = ensure_gateup_smem(smem);
        if (rc != RM_OK) return rc == RM_ERR_SHAPE ? RM_ERR_UNSUPPORTED : rc;      // H beyond what this kernel can stage
    }
    int kcap = a.count ? (int)(a.list_cap < (int64_t)g.I ? a.list_cap : (int64_t)g.I) : g.I;
    dim3 g1((kcap + GU_WARPS - 1) / GU_WARPS, a.B);
    ref_gateup_kernel<<<g1, GU_WARPS * 32, smem, s>>>(a, g, x, h, ctx->d_status);
    ctx->launches++;
    dim3 g2((g.H / 2 + DN_THREADS - 1) / DN_THREADS, (a.T + DN_TOK - 1) / DN_TOK, a.B);
    ref_down_kernel<<<g2, DN_THREADS, 0, s>>>(a, g, h, ctx->d_status);
    ctx->launches++;
    RM_CUDA_TRY(cudaGetLastError());
    return RM_OK;
}


// ---------------------------------------------------------------------------------------------------------------
// rm_sparse_mlp_static: the one-layer masked MLP for callers that must not allocate.
//
// The compact hidden activations h [T, I] that the gate/up kernel hands to the down kernel normally live in the
// caller's workspace.  Here they live in a fixed 4 MiB array inside the library image, so the call needs no context
// (rm_create allocates), no workspace and no allocator of any kind.  The array is shared by every call on a device.
namespace {

constexpr size_t RM_STATIC_H_FLOATS = (size_t)1 << 20;          // T * I <= 1,048,576 (e.g. T = 64, I = 16384)
static __device__ __align__(256) float g_static_h[RM_STATIC_H_FLOATS];

constexpr int RM_STATIC_MAX_DEVICES = 64;
std::mutex g_static_mutex;
float* g_static_h_addr[RM_STATIC_MAX_DEVICES] = {};             // device address of g_static_h, per device

}  // namespace

extern "C" int rm_sparse_mlp_static(const void* packed_layer, const void* x, const float* residual,
                                    const int32_t* idx, const int32_t* count_dev, float* y, int T, int H, int I,
                                    rm_stream_t stream) {
    if (!packed_layer || !x || !y || T < 0 || H < 64 || I < 1) return RM_ERR_INVALID_ARG;
    if (idx && !count_dev) return RM_ERR_INVALID_ARG;
    if (H % 64 != 0) return RM_ERR_SHAPE;
    if ((size_t)T * (size_t)I > RM_STATIC_H_FLOATS) return RM_ERR_SHAPE;      // beyond the built-in scratch
    for (const void* p : {packed_layer, x, (const void*)residual, (const void*)idx, (const void*)y})
        if (p && !rm_aligned16(p)) return RM_ERR_ALIGN;
    if (T == 0) return RM_OK;

    int dev = -1;
    RM_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= RM_STATIC_MAX_DEVICES) return RM_ERR_UNSUPPORTED;
    const size_t smem = (size_t)GU_WARPS * 2 * H * sizeof(__nv_bfloat16);
    {
        const int rc = ensure_gateup_smem(smem);                  // RM_ERR_SHAPE: H above 7232 does not fit a CTA's shared memory
        if (rc != RM_OK) return rc;
    }
    float* h = nullptr;
    {
        // Once per device, with that device current: ask the runtime where the array lives on this device.  In host
        // code the symbol itself is only a stand-in; handing it to a kernel would not be a device address.
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_h_addr[dev]) {
            float* p = nullptr;
            if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_h) != cudaSuccess || !p) return RM_ERR_CUDA;
            g_static_h_addr[dev] = p;
        }
        h = g_static_h_addr[dev];
    }

    rm_geom g{};
    g.L = 1;
    g.H = H;
    g.I = I;
    g.Hs = H / RM_NS;
    rm_layer_args a{};
    a.packed = static_cast<const __nv_bfloat16*>(packed_layer);
    a.x = static_cast<const __nv_bfloat16*>(x);
    a.r_in = residual;
    a.r_out = y;
    a.idx = idx;
    a.count = count_dev;                                           // with idx NULL: the leading count neurons, as in rm_sparse_mlp
    a.idx_stride = I;
    a.list_cap = I;
    a.count_stride = 1;
    a.B = 1;
    a.T = T;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Nothing in the scratch has to start at zero: the gate/up kernel writes h[t, j] for every token and every
    // list position j < count before the down kernel reads exactly those entries.
    dim3 g1((I + GU_WARPS - 1) / GU_WARPS, 1);
    ref_gateup_kernel<<<g1, GU_WARPS * 32, smem, s>>>(a, g, a.x, h, nullptr);
    dim3 g2((H / 2 + DN_THREADS - 1) / DN_THREADS, (T + DN_TOK - 1) / DN_TOK, 1);
    ref_down_kernel<<<g2, DN_THREADS, 0, s>>>(a, g, h, nullptr);
    RM_CUDA_TRY(cudaGetLastError());
    return RM_OK;
}
