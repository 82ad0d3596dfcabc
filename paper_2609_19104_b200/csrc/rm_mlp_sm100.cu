// Fused masked gated-MLP layer for sm_100a: one kernel per layer, thread-block clusters of 8 CTAs.
//
// Decomposition.  A cluster owns a contiguous range of the active neurons of a layer and walks it in tiles of 64
// neurons.  CTA j of the cluster owns column slice j (Hs = H/8 columns) of the model dimension for BOTH
// projections:
//   gate/up : D1[128 x T] = [64 gate rows ; 64 up rows](slice j) . x(slice j)^T      partial over the H split
//   exchange: partial sums are reduce-scattered through distributed shared memory (CTA o receives the rows of
//             neurons 8o..8o+7), the owner applies GeLU-tanh(g) * u, and broadcasts h (bf16) to the 8 CTAs
//   down    : D2[Hs x T] += Wd(slice j, tile)^T-as-MN-major . h^T                   accumulated over tiles in TMEM
// so a neuron's 3*Hs*2 contiguous bytes are read exactly once by exactly one CTA, x is never replicated inside a
// cluster, and h never leaves the chip.  Both products run on the 5th-generation tensor cores (tcgen05.mma,
// accumulators in tensor memory); the gathered rows are placed by 16-byte cp.async directly into the 128-byte
// swizzled operand layout.  At the end of an episode each CTA adds its [T x Hs] partial of y to the fp32 residual
// stream with red.global.add; the residual itself is added by one designated cluster per episode.
//
// Layers are chained with programmatic dependent launch: a layer's CTAs become resident, set up and trigger their
// dependents early, and wait (griddepcontrol.wait) for the previous layer's atomics before touching activations.
#include <cstdio>
#include <cstdlib>

#include "rm_common.cuh"
#include "rm_sm100.cuh"

using namespace sm100;

// Optional phase timing (build with -DRM_PHASE_TIMING): thread 0 of every CTA stamps clock64() at phase
// boundaries of its first tile into a device buffer that rm_debug_phase_times copies out.
#ifdef RM_PHASE_TIMING
__device__ long long g_phase_stamps[256 * 32];
#define RM_STAMP(k)                                                                           \
    do {                                                                                      \
        if (threadIdx.x == 0 && blockIdx.x < 256 && stamp_ok) g_phase_stamps[blockIdx.x * 32 + (k)] = clock64(); \
    } while (0)
#else
#define RM_STAMP(k) do { } while (0)
#endif

namespace {

constexpr int FT = 256;            // threads per CTA
constexpr int CS = 8;              // CTAs per cluster == column slices
constexpr int NT = 64;             // neurons per tile
constexpr int MAXB = 64;           // episodes per call on this path

struct FusedArgs {
    const __nv_bfloat16* packed;
    const __nv_bfloat16* x;        // [B,T,H] bf16, or NULL: x = bf16(RMSNorm(r_in))
    const float* r_in;             // [B,T,H] fp32 (norm source and residual)
    float* r_out;                  // [B,T,H] fp32, accumulated with atomics (pre-initialised by the caller)
    float* zero_buf;               // nullable: [B,T,H] floats this launch clears for a later layer
    const int32_t* idx;
    const int32_t* count;
    int64_t idx_stride, list_cap, count_stride;
    float* record;
    int64_t record_stride;
    const float* record_scale;
    int B, T, H, I;
    int add_residual;              // a designated cluster per episode adds r_in into r_out
    int npc_target;                // neurons per cluster aimed for when spreading a layer over clusters
    int* status;
};

template <int NTOK, int HS>
struct Smem {
    static constexpr int KB = HS / 64;                       // 64-column (128-byte) blocks per slice
    static constexpr int X_BYTES = KB * NTOK * 128;
    static constexpr int GU_BYTES = KB * 128 * 128;
    static constexpr int DN_BYTES = KB * NT * 128;
    static constexpr int HT_BYTES = NTOK * 128;
    static constexpr int P_ROW = NTOK + 4;                   // padded row (floats) of the partial-sum buffer
    static constexpr int P_BYTES = CS * 16 * P_ROW * 4;
    static constexpr int OFF_X = 0;
    static constexpr int OFF_GU = OFF_X + X_BYTES;
    static constexpr int OFF_DN = OFF_GU + GU_BYTES;
    static constexpr int OFF_HT = OFF_DN + DN_BYTES;
    static constexpr int OFF_P = OFF_HT + HT_BYTES;
    static constexpr int OFF_HS = OFF_P + P_BYTES;           // [NTOK] x 16 B: this CTA's 8 neurons per token
    static constexpr int OFF_SS = OFF_HS + NTOK * 16;        // [CS][64] floats: row sums of squares per source CTA
    static constexpr int OFF_N = OFF_SS + CS * 64 * 4;       // [64] neuron ids of the tile
    static constexpr int OFF_PREF = OFF_N + NT * 4;          // [MAXB+1] prefix of the per-episode counts
    static constexpr int OFF_BAR = OFF_PREF + (MAXB + 1) * 4 + 4;   // 8-byte aligned: two mbarriers, tmem pointer
    static constexpr int TOTAL = OFF_BAR + 32;
    static constexpr int TMEM_COLS_USED = NTOK + (HS / 128) * NTOK;
    static constexpr int TMEM_COLS = TMEM_COLS_USED <= 32 ? 32 : TMEM_COLS_USED <= 64 ? 64 :
                                     TMEM_COLS_USED <= 128 ? 128 : TMEM_COLS_USED <= 256 ? 256 : 512;
};

__device__ __forceinline__ uint4 pack8(const float* v, float s) {
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0] * s, v[1] * s), b = __floats2bfloat162_rn(v[2] * s, v[3] * s);
    __nv_bfloat162 c = __floats2bfloat162_rn(v[4] * s, v[5] * s), d = __floats2bfloat162_rn(v[6] * s, v[7] * s);
    uint4 r;
    r.x = *reinterpret_cast<uint32_t*>(&a);
    r.y = *reinterpret_cast<uint32_t*>(&b);
    r.z = *reinterpret_cast<uint32_t*>(&c);
    r.w = *reinterpret_cast<uint32_t*>(&d);
    return r;
}

template <int NTOK, int HS>
__global__ void __launch_bounds__(FT, (HS == 128 ? 2 : 1)) fused_layer_kernel(const FusedArgs a) {
    using S = Smem<NTOK, HS>;
    constexpr int KB = S::KB;
    extern __shared__ unsigned char smem_dyn[];
    // 1024-byte alignment: the 128-byte swizzle is a function of absolute shared-memory address bits
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* gbase = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t sX = base + S::OFF_X, sGU = base + S::OFF_GU, sDN = base + S::OFF_DN, sHT = base + S::OFF_HT;
    const uint32_t sP = base + S::OFF_P, sSS = base + S::OFF_SS;
    float* gP = reinterpret_cast<float*>(gbase + S::OFF_P);
    uint4* gHS = reinterpret_cast<uint4*>(gbase + S::OFF_HS);
    float* gSS = reinterpret_cast<float*>(gbase + S::OFF_SS);
    int* gN = reinterpret_cast<int*>(gbase + S::OFF_N);
    int* gPref = reinterpret_cast<int*>(gbase + S::OFF_PREF);
    const uint32_t bar_gu = base + S::OFF_BAR, bar_dn = bar_gu + 8, s_tmem = bar_gu + 16;
    volatile uint32_t* g_tmem = reinterpret_cast<volatile uint32_t*>(gbase + S::OFF_BAR + 16);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef RM_PHASE_TIMING
    bool stamp_ok = true;
#endif
    RM_STAMP(0);
    const int j = (int)cluster_ctarank();
    const int cid = (int)cluster_id_x(), NC = (int)cluster_count_x();
    const int H = a.H, T = a.T;

    // ---- set-up: barriers, tensor memory, per-episode counts
    if (tid == 0) {
        mbar_init(bar_gu, 1);
        mbar_init(bar_dn, 1);
        fence_mbar_init();
        int acc = 0;
        const int cap = (int)(a.list_cap < (int64_t)a.I ? a.list_cap : (int64_t)a.I);
        for (int b = 0; b < a.B; ++b) {
            int c = a.I;                   // dense: every neuron
            if (a.idx) {
                c = a.count[(size_t)b * a.count_stride];
                if (c < 0 || c > cap) { rm_set_status(a.status, RM_ERR_INDEX); c = c < 0 ? 0 : cap; }
            }
            gPref[b] = acc;
            acc += c;
        }
        gPref[a.B] = acc;
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(s_tmem, S::TMEM_COLS);
    }
    tc_fence_before();
    cluster_sync();                        // peers' shared memory and barriers are live from here on
    tc_fence_after();
    const uint32_t tmem_d1 = *g_tmem;
    const uint32_t tmem_d2 = tmem_d1 + NTOK;

    RM_STAMP(1);
    pdl_launch_dependents();               // the next layer may become resident and set up

    const int total = gPref[a.B];
    int n_active = (total + a.npc_target - 1) / a.npc_target;
    n_active = n_active < 1 ? 1 : (n_active > NC ? NC : n_active);
    const long long g0 = cid < n_active ? (long long)cid * total / n_active : 0;
    const long long g1 = cid < n_active ? (long long)(cid + 1) * total / n_active : 0;

    pdl_wait();                            // the previous layer's output is complete and visible
    RM_STAMP(2);

    // ---- duties that do not depend on the neuron range
    if (a.zero_buf) {
        float4* z = reinterpret_cast<float4*>(a.zero_buf);
        const size_t n4 = (size_t)a.B * T * H / 4;
        for (size_t i = (size_t)blockIdx.x * FT + tid; i < n4; i += (size_t)gridDim.x * FT)
            z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (a.add_residual) {
        for (int b = cid; b < a.B; b += NC) {
            for (int i = tid; i < T * (HS / 4); i += FT) {
                const int t = i / (HS / 4), c4 = i - t * (HS / 4);
                const size_t o = ((size_t)b * T + t) * H + (size_t)j * HS + c4 * 4;
                const float4 v = *reinterpret_cast<const float4*>(a.r_in + o);
                atomicAdd(a.r_out + o, v.x);
                atomicAdd(a.r_out + o + 1, v.y);
                atomicAdd(a.r_out + o + 2, v.z);
                atomicAdd(a.r_out + o + 3, v.w);
            }
        }
    }

    RM_STAMP(3);
    uint32_t par_gu = 0, par_dn = 0;
    bool dn_pending = false;
    constexpr uint32_t IDESC_GU = idesc_bf16_f32(128, NTOK, false, false);
    constexpr uint32_t IDESC_DN = idesc_bf16_f32(128, NTOK, true, false);

    for (int b = 0; b < a.B; ++b) {
        const long long s0 = gPref[b], s1 = gPref[b + 1];
        const int lo = (int)((g0 > s0 ? g0 : s0) - s0), hi = (int)((g1 < s1 ? g1 : s1) - s0);
        if (lo >= hi) continue;            // uniform across the cluster

        // ---- x slice of episode b -> bf16, 128-byte-swizzled K-major operand tile
        {
            constexpr int PARTS = FT / NTOK;               // threads per token row
            constexpr int CPP = HS / PARTS;                // columns per thread
            const int t = tid / PARTS, part = tid % PARTS;
            float v[CPP];
            if (a.x) {
                if (t < T) {
                    const uint4* src = reinterpret_cast<const uint4*>(a.x + ((size_t)b * T + t) * H + (size_t)j * HS + part * CPP);
#pragma unroll
                    for (int i = 0; i < CPP / 8; ++i) {
                        const uint4 u = src[i];
                        const int k = part * CPP + i * 8;
                        *reinterpret_cast<uint4*>(gbase + S::OFF_X + (k >> 6) * (NTOK * 128) + t * 128 +
                                                  ((((k & 63) >> 3) ^ (t & 7)) << 4)) = u;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < CPP / 8; ++i) {
                        const int k = part * CPP + i * 8;
                        *reinterpret_cast<uint4*>(gbase + S::OFF_X + (k >> 6) * (NTOK * 128) + t * 128 +
                                                  ((((k & 63) >> 3) ^ (t & 7)) << 4)) = make_uint4(0, 0, 0, 0);
                    }
                }
            } else {
                float ss = 0.f;
                if (t < T) {
                    const float4* src = reinterpret_cast<const float4*>(a.r_in + ((size_t)b * T + t) * H + (size_t)j * HS + part * CPP);
#pragma unroll
                    for (int i = 0; i < CPP / 4; ++i) {
                        const float4 f = src[i];
                        v[4 * i] = f.x; v[4 * i + 1] = f.y; v[4 * i + 2] = f.z; v[4 * i + 3] = f.w;
                        ss = fmaf(f.x, f.x, ss); ss = fmaf(f.y, f.y, ss); ss = fmaf(f.z, f.z, ss); ss = fmaf(f.w, f.w, ss);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < CPP; ++i) v[i] = 0.f;
                }
#pragma unroll
                for (int d = 1; d < PARTS; d <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
                if (part == 0) {
#pragma unroll
                    for (int dst = 0; dst < CS; ++dst) st_cluster_f32(map_to_rank(sSS + (j * 64 + t) * 4, dst), ss);
                }
                cluster_sync();
                float tot = 0.f;
#pragma unroll
                for (int src = 0; src < CS; ++src) tot += gSS[src * 64 + t];
                const float inv = 1.0f / sqrtf(tot / (float)H + 1e-6f);
#pragma unroll
                for (int i = 0; i < CPP / 8; ++i) {
                    const int k = part * CPP + i * 8;
                    *reinterpret_cast<uint4*>(gbase + S::OFF_X + (k >> 6) * (NTOK * 128) + t * 128 +
                                              ((((k & 63) >> 3) ^ (t & 7)) << 4)) = pack8(v + 8 * i, inv);
                }
            }
            fence_proxy_async();
        }
        RM_STAMP(4);

        for (int p0 = lo; p0 < hi; p0 += NT) {
            const int nvalid = (hi - p0) < NT ? (hi - p0) : NT;
            if (dn_pending) {              // the previous down MMA still reads the DN and HT tiles
                if (!mbar_wait(bar_dn, par_dn)) rm_set_status(a.status, RM_ERR_TIMEOUT);
                par_dn ^= 1;
                dn_pending = false;
            }
            if (tid < NT) {
                int n = -1;
                if (tid < nvalid) {
                    n = a.idx ? a.idx[(size_t)b * a.idx_stride + p0 + tid] : p0 + tid;
                    if (n < 0 || n >= a.I) { rm_set_status(a.status, RM_ERR_INDEX); n = -1; }
                }
                gN[tid] = n;
            }
            __syncthreads();

            // ---- gather this CTA's pieces of the tile: per neuron [gate Hs | up Hs | down Hs] contiguous
            const __nv_bfloat16* slice = a.packed + (size_t)j * 3 * HS;
#pragma unroll
            for (int it = 0; it < KB * 4; ++it) {
                const int i = it * FT + tid;
                const int kb = i >> 10, rr = (i >> 3) & 127, ch = i & 7;
                const int n = gN[rr & 63];
                const __nv_bfloat16* src = slice + (size_t)(n < 0 ? 0 : n) * 3 * H + (rr >> 6) * HS + kb * 64 + ch * 8;
                cp_async16(sGU + kb * 16384 + rr * 128 + ((ch ^ (rr & 7)) << 4), src, n >= 0);
            }
#pragma unroll
            for (int it = 0; it < KB * 2; ++it) {
                const int i = it * FT + tid;
                const int cb = i >> 9, q = (i >> 3) & 63, ch = i & 7;
                const int n = gN[q];
                const __nv_bfloat16* src = slice + (size_t)(n < 0 ? 0 : n) * 3 * H + 2 * HS + cb * 64 + ch * 8;
                cp_async16(sDN + cb * 8192 + q * 128 + ((ch ^ (q & 7)) << 4), src, n >= 0);
            }
            cp_async_commit();
            RM_STAMP(5);
            cp_async_wait<0>();
            fence_proxy_async();
            __syncthreads();
            RM_STAMP(6);

            // ---- gate/up partial products over this CTA's column slice
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        mma_bf16_ss(tmem_d1, smem_desc_sw128(sGU + kb * 16384 + ks * 32, 16, 1024),
                                    smem_desc_sw128(sX + kb * (NTOK * 128) + ks * 32, 16, 1024), IDESC_GU, (kb | ks) != 0);
                mma_commit(bar_gu);
            }
            if (!mbar_wait(bar_gu, par_gu)) rm_set_status(a.status, RM_ERR_TIMEOUT);
            par_gu ^= 1;
            tc_fence_after();
            RM_STAMP(7);

            // ---- reduce-scatter: row m of D1 (gate or up of tile neuron q) goes to the CTA that owns q
            for (int c0 = (warp >> 2) * 32; c0 < NTOK; c0 += 64) {
                float v[32];
                const int m = (warp & 3) * 32 + lane;
                tmem_ld32(tmem_d1 + ((uint32_t)((warp & 3) * 32) << 16) + c0, v);
                const int q = m & 63;
                const uint32_t dst = map_to_rank(sP + ((j * 16 + (m >> 6) * 8 + (q & 7)) * S::P_ROW + c0) * 4, q >> 3);
#pragma unroll
                for (int i = 0; i < 8; ++i) st_cluster_v4(dst + i * 16, v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            }
            tc_fence_before();
            RM_STAMP(8);
            cluster_sync();                // (1) all partial sums have landed
            RM_STAMP(9);

            // ---- owner: sum the 8 partials, GeLU-tanh(g) * u, activation record, bf16 h
            {
                constexpr int TPL = NTOK / 32;             // tokens per lane
                const int ql = warp;                       // local neuron 0..7 (tile neuron 8j + ql)
                float g[TPL], u[TPL];
#pragma unroll
                for (int i = 0; i < TPL; ++i) g[i] = u[i] = 0.f;
#pragma unroll
                for (int src = 0; src < CS; ++src) {
                    const float* pg = gP + (src * 16 + ql) * S::P_ROW + lane * TPL;
                    const float* pu = gP + (src * 16 + 8 + ql) * S::P_ROW + lane * TPL;
#pragma unroll
                    for (int i = 0; i < TPL; ++i) { g[i] += pg[i]; u[i] += pu[i]; }
                }
                float rec = 0.f;
                __nv_bfloat16* hs = reinterpret_cast<__nv_bfloat16*>(gHS);
#pragma unroll
                for (int i = 0; i < TPL; ++i) {
                    const float h = rm_gelu_tanh(g[i]) * u[i];
                    rec += fabsf(h);
                    hs[(lane * TPL + i) * 8 + ql] = __float2bfloat16_rn(h);
                }
                if (a.record) {
#pragma unroll
                    for (int d = 16; d > 0; d >>= 1) rec += __shfl_xor_sync(0xffffffffu, rec, d);
                    const int n = gN[j * 8 + ql];
                    if (lane == 0 && n >= 0)
                        a.record[(size_t)b * a.record_stride + n] = a.record_scale ? rec * a.record_scale[n] : rec;
                }
            }
            __syncthreads();
            // ---- all-gather h: token row t, 16-byte chunk j (neurons 8j..8j+7) of every CTA's K-major h tile
            for (int i = tid; i < NTOK * CS; i += FT) {
                const int t = i % NTOK, dst = i / NTOK;
                st_cluster_v4u(map_to_rank(sHT + t * 128 + ((j ^ (t & 7)) << 4), dst), gHS[t]);
            }
            fence_proxy_async();
            RM_STAMP(10);
            cluster_sync();                // (2) h of the whole tile is present in every CTA
            RM_STAMP(11);

            // ---- down projection of the tile, accumulated in tensor memory across the episode's tiles
            if (tid == 0) {
                fence_proxy_async();
                tc_fence_after();
#pragma unroll
                for (int mm = 0; mm < HS / 128; ++mm)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        mma_bf16_ss(tmem_d2 + mm * NTOK, smem_desc_sw128(sDN + mm * 16384 + ks * 2048, 8192, 1024),
                                    smem_desc_sw128(sHT + ks * 32, 16, 1024), IDESC_DN, !(p0 == lo && ks == 0));
                mma_commit(bar_dn);
            }
            dn_pending = true;
            RM_STAMP(12);
#ifdef RM_PHASE_TIMING
            stamp_ok = false;              // first tile only
#endif
        }
#ifdef RM_PHASE_TIMING
        stamp_ok = true;
#endif

        // ---- add this CTA's [T x Hs] partial of y to the residual stream
        if (!mbar_wait(bar_dn, par_dn)) rm_set_status(a.status, RM_ERR_TIMEOUT);
        par_dn ^= 1;
        dn_pending = false;
        tc_fence_after();
        RM_STAMP(13);
#pragma unroll
        for (int mm = 0; mm < HS / 128; ++mm) {
            for (int c0 = (warp >> 2) * 32; c0 < NTOK; c0 += 64) {
                float v[32];
                tmem_ld32(tmem_d2 + mm * NTOK + ((uint32_t)((warp & 3) * 32) << 16) + c0, v);
                float* dst = a.r_out + (size_t)b * T * H + (size_t)j * HS + mm * 128 + (warp & 3) * 32 + lane;
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (c0 + i < T) atomicAdd(dst + (size_t)(c0 + i) * H, v[i]);
            }
        }
        tc_fence_before();
        __syncthreads();
        RM_STAMP(14);
    }

    // ---- teardown: nobody may still be writing into this CTA's shared memory; release tensor memory
    tc_fence_before();
    cluster_sync();
    if (warp == 0) tmem_dealloc(tmem_d1, S::TMEM_COLS);
    RM_STAMP(15);
}

template <int NTOK, int HS>
int launch_fused(rm_ctx* ctx, const FusedArgs& a, int n_clusters, bool pdl, cudaStream_t s) {
    using S = Smem<NTOK, HS>;
    auto kern = fused_layer_kernel<NTOK, HS>;
    const int smem = S::TOTAL + 1024;
    static bool configured = false;
    if (!configured) {
        RM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_clusters * CS);
    cfg.blockDim = dim3(FT);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = CS;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 2 : 1;
    RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, a));
    ctx->launches++;
    return RM_OK;
}

template <int NTOK, int HS>
int max_clusters(int* out, int* blocks_per_sm) {
    using S = Smem<NTOK, HS>;
    auto kern = fused_layer_kernel<NTOK, HS>;
    const int smem = S::TOTAL + 1024;
    RM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CS * 64);
    cfg.blockDim = dim3(FT);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = CS;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    RM_CUDA_TRY(cudaOccupancyMaxActiveClusters(out, kern, &cfg));
    if (blocks_per_sm) RM_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, kern, FT, smem));
    if (getenv("RM_DEBUG_OCC")) {
        cudaFuncAttributes fa;
        cudaFuncGetAttributes(&fa, kern);
        int b2 = -1;
        for (int sm : {16 * 1024, 48 * 1024, 100 * 1024}) {
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b2, kern, FT, sm);
            fprintf(stderr, "  smem %d -> blocks %d\n", sm, b2);
        }
        cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b2, kern, FT, smem);
        fprintf(stderr, "  with carveout 100: smem %d -> blocks %d\n", smem, b2);
        fprintf(stderr, "fused<%d,%d>: regs %d static smem %zu maxdyn %d local %zu smem req %d blocks@100KB %d\n", NTOK, HS,
                fa.numRegs, fa.sharedSizeBytes, fa.maxDynamicSharedSizeBytes, fa.localSizeBytes, smem, b2);
    }
    return RM_OK;
}

}  // namespace

int rm_fused_debug_stamps(long long* host_out, int n) {
#ifdef RM_PHASE_TIMING
    if (n > 256 * 32) n = 256 * 32;
    return cudaMemcpyFromSymbol(host_out, g_phase_stamps, sizeof(long long) * n) == cudaSuccess ? RM_OK : RM_ERR_CUDA;
#else
    (void)host_out; (void)n;
    return RM_ERR_UNSUPPORTED;
#endif
}

bool rm_fused_supported(const rm_ctx* ctx, int B, int T) {
    const int H = ctx->g.H;
    return (H == 1024 || H == 2048) && T >= 1 && T <= 64 && B >= 1 && B <= MAXB && ctx->fused_clusters > 0;
}

int rm_fused_init(rm_ctx* ctx) {
    ctx->fused_clusters = 0;
    int n = 0, rc = RM_OK;
    if (ctx->g.H == 1024) rc = max_clusters<64, 128>(&n, &ctx->fused_blocks_per_sm);
    else if (ctx->g.H == 2048) rc = max_clusters<64, 256>(&n, &ctx->fused_blocks_per_sm);
    else return RM_OK;
    if (rc != RM_OK) return rc;
    ctx->fused_clusters = n;
    return RM_OK;
}

int rm_launch_layer_fused(rm_ctx* ctx, const rm_layer_args& la, float* zero_buf, bool add_residual, bool pdl,
                          cudaStream_t s) {
    FusedArgs a{};
    a.packed = la.packed;
    a.x = la.x;
    a.r_in = la.r_in;
    a.r_out = la.r_out;
    a.zero_buf = zero_buf;
    a.idx = la.idx;
    a.count = la.count;
    a.idx_stride = la.idx_stride;
    a.list_cap = la.list_cap;
    a.count_stride = la.count_stride;
    a.record = la.record;
    a.record_stride = la.record_stride;
    a.record_scale = la.record_scale;
    a.B = la.B;
    a.T = la.T;
    a.H = ctx->g.H;
    a.I = ctx->g.I;
    a.add_residual = add_residual ? 1 : 0;
    a.npc_target = ctx->npc_target;
    a.status = ctx->d_status;
    // Clusters per launch: all co-resident slots, or -- when the caller told us how many neurons to expect -- just
    // enough for them, which leaves slots free for the next layer's CTAs to become resident early.
    int nc = ctx->fused_clusters;
    if (ctx->count_hint > 0) {
        long long want = ((long long)ctx->count_hint * la.B + ctx->npc_target - 1) / ctx->npc_target;
        if (want < 1) want = 1;
        if (want < nc) nc = (int)want;
    }
    if (ctx->max_clusters_override > 0 && nc > ctx->max_clusters_override) nc = ctx->max_clusters_override;
    const bool small_t = la.T <= 32;
    if (ctx->g.H == 1024) return small_t ? launch_fused<32, 128>(ctx, a, nc, pdl, s) : launch_fused<64, 128>(ctx, a, nc, pdl, s);
    return small_t ? launch_fused<32, 256>(ctx, a, nc, pdl, s) : launch_fused<64, 256>(ctx, a, nc, pdl, s);
}
