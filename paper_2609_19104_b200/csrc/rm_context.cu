// Context Cache: visual-token selective recomputation of a VLM FFN (Sec. 4.1 "Visual-Token Recomputation").
//   Eq. 2   drift score d_p = RMS(x_p - xref_p) / max(RMS(x_p), 1e-6) per visual row
//   Eq. 3   y_hat_p = F(x_p) for the selected rows (and the rows that are always recomputed), else the reference output
// F is the dense gated FFN, F(x) = Wd (gelu_tanh(Wg x) * (Wu x)).  With a few hundred rows against 100 M weights this
// is a pair of dense contractions at the ridge of the roofline, so it runs on the tensor cores with every operand
// block arriving as one cp.async.bulk.tensor box:
//   gather  : Xc[r,:] = x[rows[r],:]                                   (R_pad rows, zero beyond the list)
//   phase A : H1[r, n] = bf16(gelu_tanh(<Xc_r, Wg_n>) * <Xc_r, Wu_n>)  one CTA per 128 neurons, K = H
//   phase B : Yp[s][r, c] = sum over the s-th slice of n of H1[r, n] Wd[c, n]   one CTA per (128 columns, K slice)
//   scatter : y_out = y_ref, then y_out[rows[r], :] = sum_s Yp[s][r, :]
// Both products are D[128 x NR] (+)= A[128 x 64] B[NR x 64]^T per stage: A = weight rows (K contiguous, as the model
// stores them), B = activation rows, fp32 accumulators in tensor memory (phase A holds two, gate and up: all 512 columns
// at NR = 256).
#include <cuda.h>

#include <mutex>

#include "rm_common.cuh"
#include "rm_sm100.cuh"

using namespace sm100;

namespace {

constexpr int CT = 192;                // threads: epilogue warps 0-3, loader warp 4 (one lane), issuer warp 5 (one lane)

__device__ __forceinline__ void tma_box(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t mbar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(mbar) : "memory");
}

// ---------------------------------------------------------------- Eq. 2: one warp per row
__global__ void __launch_bounds__(256) drift_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ xr,
                                                    int P, int H, float* __restrict__ score) {
    pdl_launch_dependents();               // the selection kernel behind this one may set up
    const int p = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (p >= P) return;
    const uint4* a = reinterpret_cast<const uint4*>(x + (size_t)p * H);
    const uint4* b = reinterpret_cast<const uint4*>(xr + (size_t)p * H);
    float sd = 0.f, sx = 0.f;
    for (int e = lane; e < H / 8; e += 32) {
        const uint4 ua = a[e], ub = b[e];
        const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&ua);
        const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&ub);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 fa = __bfloat1622float2(pa[i]), fb = __bfloat1622float2(pb[i]);
            const float d0 = fa.x - fb.x, d1 = fa.y - fb.y;
            sd = fmaf(d0, d0, sd); sd = fmaf(d1, d1, sd);
            sx = fmaf(fa.x, fa.x, sx); sx = fmaf(fa.y, fa.y, sx);
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        sd += __shfl_xor_sync(0xffffffffu, sd, d);
        sx += __shfl_xor_sync(0xffffffffu, sx, d);
    }
    if (lane == 0) score[p] = sqrtf(sd / (float)H) / fmaxf(sqrtf(sx / (float)H), 1e-6f);
}

// ---------------------------------------------------------------- gather of the rows to recompute
// The rows to recompute form one sequence q = 0, 1, ...: q < count is the visual row rows[q], count <= q < count + S the
// always-recomputed row P + (q - count).  A call holds at most `cap` of them (a longer list is cut and reported); one
// pass of the kernels handles the window q_lo <= q < q_lo + r_pad, compact row r = q - q_lo; rows beyond the sequence
// are zero.
__device__ __forceinline__ int ctx_count(const int32_t* count, int P, int S, int cap, bool* bad) {
    int c = *count;
    *bad = c < 0 || c > P || c + S > cap;
    if (*bad) c = c < 0 ? 0 : (P < cap - S ? P : cap - S);
    return c;
}
__global__ void __launch_bounds__(256) ctx_gather_kernel(const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ rows,
                                                         const int32_t* __restrict__ count, int P, int S, int H, int r_pad,
                                                         int q_lo, int cap, __nv_bfloat16* __restrict__ xc, int* status) {
    pdl_launch_dependents();               // the first product may start now: its weight loads need nothing from here
    pdl_wait();                            // the row list comes from the kernel in front
    const int r = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (r >= r_pad) return;
    bool bad;
    const int c = ctx_count(count, P, S, cap, &bad);
    if (bad && r == 0 && lane == 0) rm_set_status(status, RM_ERR_INDEX);
    const int q = q_lo + r;
    int src = -1;
    if (q < c) {
        src = rows[q];
        if (src < 0 || src >= P) { if (lane == 0) rm_set_status(status, RM_ERR_INDEX); src = -1; }
    } else if (q < c + S) {
        src = P + (q - c);
    }
    uint4* d = reinterpret_cast<uint4*>(xc + (size_t)r * H);
    const uint4* s = src >= 0 ? reinterpret_cast<const uint4*>(x + (size_t)src * H) : nullptr;
    for (int e = lane; e < H / 8; e += 32) d[e] = s ? s[e] : make_uint4(0, 0, 0, 0);
}

// ---------------------------------------------------------------- scatter: recomputed rows and kept reference rows
// CTAs 0 .. r_pad-1: output row of recomputed row r = sum of the K slices.  CTAs r_pad .. r_pad+P-1: visual row p keeps
// its reference output unless it is in the (ascending) list.
__global__ void __launch_bounds__(256) ctx_scatter_kernel(const float* __restrict__ yp, int ksplit, int r_pad,
                                                          const int32_t* __restrict__ rows, const int32_t* __restrict__ count,
                                                          int P, int S, int H, int q_lo, int cap, const float* __restrict__ y_ref,
                                                          float* __restrict__ y_out) {
    pdl_wait();                            // the partial products come from the kernel in front
    bool bad;
    const int c = ctx_count(count, P, S, cap, &bad);
    if ((int)blockIdx.x >= r_pad) {       // (the first pass of a call only: its grid alone has these CTAs)
        const int p = (int)blockIdx.x - r_pad;
        if (y_out == y_ref) return;
        int lo = 0, hi = c;                // is p in rows[0 .. c)?
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (rows[mid] < p) lo = mid + 1; else hi = mid;
        }
        if (lo < c && rows[lo] == p) return;
        for (int e = threadIdx.x; e < H / 4; e += blockDim.x)
            reinterpret_cast<float4*>(y_out + (size_t)p * H)[e] = reinterpret_cast<const float4*>(y_ref + (size_t)p * H)[e];
        return;
    }
    const int r = blockIdx.x, q = q_lo + r;
    int dst = -1;
    if (q < c) {
        dst = rows[q];
        if (dst >= P) dst = -1;            // a listed row must be a visual row: the gather zeroed it and recorded the error;
                                           // writing it would race with the always-recomputed row of the same number
    } else if (q < c + S) dst = P + (q - c);
    if (dst < 0 || dst >= P + S) return;
    for (int e = threadIdx.x; e < H / 4; e += blockDim.x) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < ksplit; ++s) {
            const float4 v = reinterpret_cast<const float4*>(yp + ((size_t)s * r_pad + r) * H)[e];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        reinterpret_cast<float4*>(y_out + (size_t)dst * H)[e] = acc;
    }
}

// ---------------------------------------------------------------- the two products
// DUAL (phase A): A0 = Wg rows, A1 = Wu rows of this CTA's 128 neurons over all K = H; epilogue GeLU*u -> bf16 H1.
// !DUAL (phase B): A0 = Wd rows of this CTA's 128 output columns over its K slice; epilogue fp32 partial -> Yp.
template <int NR, bool DUAL>
struct SmemCtx {
    static constexpr int A_BYTES = 128 * 128;                      // 128 rows x 64 bf16
    static constexpr int B_BYTES = NR * 128;
    static constexpr int STAGE = (DUAL ? 2 : 1) * A_BYTES + B_BYTES;
    static constexpr int NSTAGE = (200 * 1024) / STAGE > 6 ? 6 : (200 * 1024) / STAGE;
    static constexpr int OFF_STG = NSTAGE * STAGE;                 // epilogue staging: 32 rows x 256 bytes
    static constexpr int OFF_BAR = OFF_STG + 8192;
    static constexpr int TOTAL = OFF_BAR + 256 + 1024;
    static constexpr int TMEM_COLS = (DUAL ? 2 : 1) * NR < 32 ? 32 : (DUAL ? 2 : 1) * NR;
};

struct CtxGemmArgs {
    int kblocks;                       // 64-wide K blocks per CTA
    int I, H, r_pad;
    __nv_bfloat16* h1;                 // phase A output [r_pad, I]
    float* yp;                         // phase B output [ksplit, r_pad, H]
    int* status;
};

#define wait_bar(bar, parity) wait_bar_at((bar), (parity), __LINE__)

template <int NR, bool DUAL>
__global__ void __launch_bounds__(CT, 1) ctx_gemm_kernel(const CtxGemmArgs a, const __grid_constant__ CUtensorMap tmA0,
                                                         const __grid_constant__ CUtensorMap tmA1,
                                                         const __grid_constant__ CUtensorMap tmB) {
    using S = SmemCtx<NR, DUAL>;
    constexpr int NSTAGE = S::NSTAGE;
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* gbase = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t bar0 = base + S::OFF_BAR;
    auto full = [&](int s) { return bar0 + 8 * s; };
    auto empty = [&](int s) { return bar0 + 64 + 8 * s; };
    const uint32_t d_full = bar0 + 128, s_tmem = bar0 + 136;
    volatile uint32_t* g_tmem = reinterpret_cast<volatile uint32_t*>(gbase + S::OFF_BAR + 136);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < NSTAGE; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        mbar_init(d_full, 1);
        fence_mbar_init();
    }
    if (warp == 5) tmem_alloc(s_tmem, S::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *g_tmem;
    pdl_launch_dependents();

    bool gave_up = false;
    auto wait_bar_at = [&](uint32_t bar, uint32_t parity, int line) {
        if (!mbar_wait(bar, parity)) {
            rm_set_status_at(a.status, RM_ERR_TIMEOUT, (line << 12) | (int)(blockIdx.x & 0xfffu));
            gave_up = true;
        }
    };
    // this CTA's block of A rows and its K range
    const int m0 = DUAL ? (int)blockIdx.x * 128 : (int)blockIdx.x * 128;       // neurons (A) or output columns (B)
    const int kb0 = DUAL ? 0 : (int)blockIdx.y * a.kblocks;
    constexpr uint32_t IDESC = idesc_bf16_f32(128, NR, false, false);
    const uint64_t desc_k = smem_desc_sw128(0, 16, 1024);

    if (warp == 4 && lane == 0) {
        // ---- loader: the weights do not depend on the previous kernel, the activations do
        bool waited = false;
        const int pre = a.kblocks < NSTAGE ? a.kblocks : NSTAGE;
        for (int kb = 0; kb < pre; ++kb) {
            const uint32_t st = base + kb * S::STAGE;
            mbar_arrive_expect_tx(full(kb), S::STAGE);
            tma_box(st, &tmA0, (kb0 + kb) * 64, m0, full(kb));
            if (DUAL) tma_box(st + S::A_BYTES, &tmA1, (kb0 + kb) * 64, m0, full(kb));
        }
        pdl_wait();
        waited = true;
        for (int kb = 0; kb < pre; ++kb)
            tma_box(base + kb * S::STAGE + (DUAL ? 2 : 1) * S::A_BYTES, &tmB, (kb0 + kb) * 64, 0, full(kb));
        for (int kb = pre; kb < a.kblocks; ++kb) {
            const int s = kb % NSTAGE;
            wait_bar(empty(s), ((kb / NSTAGE) - 1) & 1);
            const uint32_t st = base + s * S::STAGE;
            mbar_arrive_expect_tx(full(s), S::STAGE);
            tma_box(st, &tmA0, (kb0 + kb) * 64, m0, full(s));
            if (DUAL) tma_box(st + S::A_BYTES, &tmA1, (kb0 + kb) * 64, m0, full(s));
            tma_box(st + (DUAL ? 2 : 1) * S::A_BYTES, &tmB, (kb0 + kb) * 64, 0, full(s));
        }
        (void)waited;
    } else if (warp == 5 && lane == 0) {
        // ---- issuer
        for (int kb = 0; kb < a.kblocks; ++kb) {
            const int s = kb % NSTAGE;
            const uint32_t st = base + s * S::STAGE;
            wait_bar(full(s), (kb / NSTAGE) & 1);
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const uint64_t bd = desc_k | desc_addr(st + (DUAL ? 2 : 1) * S::A_BYTES + ks * 32);
                mma_bf16_ss(tmem, desc_k | desc_addr(st + ks * 32), bd, IDESC, (kb | ks) != 0);
                if (DUAL) mma_bf16_ss(tmem + NR, desc_k | desc_addr(st + S::A_BYTES + ks * 32), bd, IDESC, (kb | ks) != 0);
            }
            mma_commit(empty(s));
        }
        mma_commit(d_full);
    } else if (warp < 4) {
        // ---- epilogue: lane = A row (neuron or output column), registers = activation rows
        const int m = tid;
        wait_bar(d_full, 0);
        tc_fence_after();
        unsigned char* stg = gbase + S::OFF_STG;
        for (int c0 = 0; c0 < NR; c0 += 32) {
            float v[32];
            tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + c0, v);
            if (DUAL) {
                float u[32];
                tmem_ld32(tmem + NR + ((uint32_t)(warp * 32) << 16) + c0, u);
                // h for 32 activation rows x this neuron -> staging [row][128 neurons] bf16, then 16-byte stores
                named_barrier(1, 128);
                // in stages over the 32 values, so that the exponentials and divisions of different rows overlap
                // (one warp per scheduler runs this; a value-by-value chain costs ~140 clocks per value)
                float e[32];
#pragma unroll
                for (int t = 0; t < 32; ++t) e[t] = __expf(-1.5957691216057308f * (v[t] + 0.044715f * v[t] * v[t] * v[t]));
#pragma unroll
                for (int t = 0; t < 32; ++t) e[t] = __fdividef(v[t], 1.0f + e[t]) * u[t];
#pragma unroll
                for (int t = 0; t < 32; ++t) reinterpret_cast<__nv_bfloat16*>(stg)[t * 128 + m] = __float2bfloat16_rn(e[t]);
                named_barrier(1, 128);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int e = m + 128 * i;                     // 512 chunks of 16 bytes: row e / 16, chunk e % 16
                    const int t = e >> 4, ch = e & 15;
                    const uint4 q = reinterpret_cast<const uint4*>(stg)[e];
                    *reinterpret_cast<uint4*>(a.h1 + (size_t)(c0 + t) * a.I + m0 + ch * 8) = q;
                }
            } else {
                float* dst = a.yp + ((size_t)blockIdx.y * a.r_pad + c0) * a.H + m0 + m;
#pragma unroll
                for (int t = 0; t < 32; ++t) dst[(size_t)t * a.H] = v[t];
            }
        }
        tc_fence_before();
    }
    tc_fence_before();
    if (__syncthreads_or(gave_up)) linger_after_timeout();
    if (warp == 5) tmem_dealloc(tmem, S::TMEM_COLS);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}
// bf16 matrix [rows, cols] row-major, boxes of box_rows x 64 columns, 128-byte swizzle
int make_map(CUtensorMap* tm, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return RM_ERR_UNSUPPORTED;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * sizeof(__nv_bfloat16)};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t es[2] = {1, 1};
    const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? RM_OK : RM_ERR_CUDA;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

template <int NR>
int run_ffn(rm_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, const __nv_bfloat16* xc, __nv_bfloat16* h1,
            float* yp, int ksplit, cudaStream_t s) {
    const int H = ctx->g.H, I = ctx->g.I;
    using SA = SmemCtx<NR, true>;
    using SB = SmemCtx<NR, false>;
    static rm_smem_configured configured = {};
    if (!configured.covers(ctx->device, SA::TOTAL)) {
        RM_CUDA_TRY(cudaFuncSetAttribute(ctx_gemm_kernel<NR, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SA::TOTAL));
        RM_CUDA_TRY(cudaFuncSetAttribute(ctx_gemm_kernel<NR, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SB::TOTAL));
        configured.set(ctx->device, SA::TOTAL);
    }
    CUtensorMap tg, tu, tx, td, th;
    int rc;
    if ((rc = make_map(&tg, Wg, I, H, 128)) != RM_OK) return rc;
    if ((rc = make_map(&tu, Wu, I, H, 128)) != RM_OK) return rc;
    if ((rc = make_map(&tx, xc, NR, H, NR)) != RM_OK) return rc;
    if ((rc = make_map(&td, Wd, H, I, 128)) != RM_OK) return rc;
    if ((rc = make_map(&th, h1, NR, I, NR)) != RM_OK) return rc;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    CtxGemmArgs a{};
    a.I = I; a.H = H; a.r_pad = NR; a.h1 = h1; a.yp = yp; a.status = ctx->d_status;
    {
        a.kblocks = H / 64;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(I / 128);
        cfg.blockDim = dim3(CT);
        cfg.dynamicSmemBytes = SA::TOTAL;
        cfg.stream = s;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, ctx_gemm_kernel<NR, true>, a, tg, tu, tx));
        ctx->launches++;
    }
    {
        a.kblocks = I / 64 / ksplit;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(H / 128, ksplit);
        cfg.blockDim = dim3(CT);
        cfg.dynamicSmemBytes = SB::TOTAL;
        cfg.stream = s;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, ctx_gemm_kernel<NR, false>, a, td, td, th));
        ctx->launches++;
    }
    return RM_OK;
}

// K slices of the second product: as many as keep about one CTA per SM, dividing the 64-wide K blocks evenly
int pick_ksplit(const rm_ctx* ctx) {
    const int col_blocks = ctx->g.H / 128, kblocks = ctx->g.I / 64;
    int best = 1;
    for (int ks = 1; ks <= 32; ++ks)
        if (kblocks % ks == 0 && col_blocks * ks <= (ctx->sm_count > 0 ? ctx->sm_count : 148)) best = ks;
    return best;
}

}  // namespace

bool rm_context_supported(const rm_ctx* ctx) { return ctx->g.H % 128 == 0 && ctx->g.I % 128 == 0; }

size_t rm_context_workspace_bytes_impl(const rm_ctx* ctx, int r_pad) {
    const size_t xc = align_up((size_t)r_pad * ctx->g.H * sizeof(__nv_bfloat16), 1024);
    const size_t h1 = align_up((size_t)r_pad * ctx->g.I * sizeof(__nv_bfloat16), 1024);
    const size_t yp = align_up((size_t)pick_ksplit(ctx) * r_pad * ctx->g.H * sizeof(float), 1024);
    return xc + h1 + yp;
}

int rm_launch_context_drift(rm_ctx* ctx, const void* x, const void* x_ref, int P, float* score, cudaStream_t s) {
    drift_kernel<<<(P + 7) / 8, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(x_ref), P,
                                            ctx->g.H, score);
    ctx->launches++;
    RM_CUDA_TRY(cudaGetLastError());
    return RM_OK;
}

int rm_launch_context_ffn(rm_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, const void* x, const int32_t* rows,
                          const int32_t* count, int P, int S, int cap, const float* y_ref, float* y_out, void* ws,
                          cudaStream_t s) {
    const int H = ctx->g.H, I = ctx->g.I;
    const int ksplit = pick_ksplit(ctx);
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    // Up to 256 rows go through the products at once; a longer sequence takes further passes over the weights (the
    // paper's own setting, 40 % of 768 visual rows plus 48 others = 356 rows, takes two).
    for (int q_lo = 0; q_lo < cap; q_lo += 256) {
        const int left = cap - q_lo;
        const int r_pad = left <= 64 ? 64 : (left <= 128 ? 128 : 256);
        char* w = static_cast<char*>(ws);
        __nv_bfloat16* xc = reinterpret_cast<__nv_bfloat16*>(w);
        w += align_up((size_t)r_pad * H * sizeof(__nv_bfloat16), 1024);
        __nv_bfloat16* h1 = reinterpret_cast<__nv_bfloat16*>(w);
        w += align_up((size_t)r_pad * I * sizeof(__nv_bfloat16), 1024);
        float* yp = reinterpret_cast<float*>(w);
        {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((r_pad + 7) / 8);
            cfg.blockDim = dim3(256);
            cfg.stream = s;
            cfg.attrs = at;
            cfg.numAttrs = 1;
            RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, ctx_gather_kernel, static_cast<const __nv_bfloat16*>(x), rows, count, P, S, H, r_pad,
                                           q_lo, cap, xc, ctx->d_status));
            ctx->launches++;
        }
        int rc = RM_ERR_SHAPE;
        if (r_pad == 64) rc = run_ffn<64>(ctx, Wg, Wu, Wd, xc, h1, yp, ksplit, s);
        else if (r_pad == 128) rc = run_ffn<128>(ctx, Wg, Wu, Wd, xc, h1, yp, ksplit, s);
        else if (r_pad == 256) rc = run_ffn<256>(ctx, Wg, Wu, Wd, xc, h1, yp, ksplit, s);
        if (rc != RM_OK) return rc;
        {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(r_pad + (q_lo == 0 ? P : 0));      // the first pass also copies the kept reference rows
            cfg.blockDim = dim3(256);
            cfg.stream = s;
            cfg.attrs = at;
            cfg.numAttrs = 1;
            RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, ctx_scatter_kernel, static_cast<const float*>(yp), ksplit, r_pad, rows, count, P, S, H,
                                           q_lo, cap, y_ref, y_out));
            ctx->launches++;
        }
    }
    return RM_OK;
}
