// Streaming variant of the masked gated MLP layer for launches with many 64-neuron tiles (dense passes, large K,
// batches): every CTA owns whole tiles, so nothing is exchanged between CTAs.
//
//   prep kernel  : x = bf16(r / sqrt(mean r^2 + 1e-6)) to global memory, and the layer's output buffer starts as a
//                  copy of r (plus gate * y_anchor in an update step of Eq. 4)
//   tile kernel  : one CTA per SM walks tiles g = cta, cta + grid, ...  For a tile it streams the gate and up rows of
//                  its 64 neurons and the matching x columns through a ring of shared-memory stages (64 columns per
//                  stage), accumulates D1[128 x T_pad] over the whole width H in tensor memory, applies GeLU-tanh(g)*u
//                  (record, Eq. 4 bookkeeping), keeps h = hi + lo (bf16 pair) in shared memory, then streams the tile's
//                  down rows 128 output columns at a time, D2 = Wd_block * h in tensor memory (two slots), and adds
//                  each finished block to the output: transposed through shared memory and added by the copy engine
//                  as one box of the [B, T, H] tensor map (two boxes in the anchor step, which also accumulates the
//                  ungated block into y_anchor).
//                  Four warps load: 16-byte cp.async gathers straight into the swizzled operand layout for index
//                  lists (they top out near 16 bytes per clock and SM), cp.async.bulk.tensor boxes of 64 neurons x 64
//                  columns for runs of consecutive neurons (one-row boxes were tried for lists and are far slower);
//                  four warps read tensor memory and do the arithmetic, one thread issues the tcgen05.mma
//                  instructions.
//
// Compared with the cluster kernels this trades the exchange latency (three hops per tile) for re-reading x from L2
// once per tile and for T*H added elements per tile; it wins when there are enough tiles to occupy the SMs.
#include <cuda.h>

#include <mutex>

#include "rm_common.cuh"
#include "rm_sm100.cuh"

using namespace sm100;

namespace {

constexpr int NT = 64;                 // neurons per tile
constexpr int MAXB = 64;               // episodes per launch
constexpr int NSTAGE = 6;
constexpr int W_BYTES = 16384;         // 128 rows (64 gate + 64 up, or 64 neurons x 2 column blocks) x 128 bytes
constexpr int STAGE = 24576;           // + x block: up to 64 token rows x 128 bytes

struct StreamArgs {
    const __nv_bfloat16* packed;
    const __nv_bfloat16* x;            // [B,T,H] bf16 (normalised)
    float* r_out;                      // [B,T,H] fp32, already holding the residual part; tiles are added to it
    const int32_t* idx;
    const int32_t* count;
    int64_t idx_stride, list_cap, count_stride;
    float* record;
    int64_t record_stride;
    const float* record_scale;
    int B, T, H, I;
    int* status;
    int anchor_mode;
    float* y_anchor;
    float* h_anchor;
    int64_t h_stride;
    const float* gate;
};

struct PrepArgs {
    const float* r_in;
    __nv_bfloat16* x;
    float* r_out;
    const float* y_anchor;             // update steps: out starts as r + gate * y_anchor
    const float* gate;
    int T, H;
};

// One CTA per token row: x row in bf16, output row = residual (+ gate * y_anchor).
__global__ void __launch_bounds__(256) stream_prep_kernel(const PrepArgs a) {
    __shared__ float part[8];
    pdl_launch_dependents();
    pdl_wait();                            // the previous layer's adds into r_in are complete
    const int row = blockIdx.x, b = row / a.T;
    const float4* src = reinterpret_cast<const float4*>(a.r_in + (size_t)row * a.H);
    const int n4 = a.H / 4;
    float4 v[2];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int e = threadIdx.x + i * 256;
        v[i] = e < n4 ? src[e] : make_float4(0.f, 0.f, 0.f, 0.f);
        ss = fmaf(v[i].x, v[i].x, ss); ss = fmaf(v[i].y, v[i].y, ss);
        ss = fmaf(v[i].z, v[i].z, ss); ss = fmaf(v[i].w, v[i].w, ss);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += part[w];
    const float inv = 1.0f / sqrtf(tot / (float)a.H + 1e-6f);
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int e = threadIdx.x + i * 256;
        if (e >= n4) continue;
        __nv_bfloat162 lo = __floats2bfloat162_rn(v[i].x * inv, v[i].y * inv);
        __nv_bfloat162 hi = __floats2bfloat162_rn(v[i].z * inv, v[i].w * inv);
        uint2 u;
        u.x = *reinterpret_cast<uint32_t*>(&lo);
        u.y = *reinterpret_cast<uint32_t*>(&hi);
        reinterpret_cast<uint2*>(a.x + (size_t)row * a.H)[e] = u;
        float4 o = v[i];
        if (a.y_anchor) {
            const float4 ya = reinterpret_cast<const float4*>(a.y_anchor + (size_t)row * a.H)[e];
            float4 g = make_float4(1.f, 1.f, 1.f, 1.f);
            if (a.gate) g = reinterpret_cast<const float4*>(a.gate + (size_t)b * a.H)[e];
            o.x = fmaf(g.x, ya.x, o.x); o.y = fmaf(g.y, ya.y, o.y); o.z = fmaf(g.z, ya.z, o.z); o.w = fmaf(g.w, ya.w, o.w);
        }
        reinterpret_cast<float4*>(a.r_out + (size_t)row * a.H)[e] = o;
    }
}

template <int NTOK>
struct SmemST {
    static constexpr int OFF_RING = 0;
    static constexpr int OFF_HT = OFF_RING + NSTAGE * STAGE;       // h tile: hi 8 KB, lo 8 KB (64 neurons x 128 bytes)
    static constexpr int OFF_Y = OFF_HT + 2 * NT * 128;            // 2 x 32 KB: GeLU exchange [2][token][neuron] fp32 (first
                                                                   // buffer), then the transposed down blocks [token][128
                                                                   // columns] fp32, alternating between the two buffers
    static constexpr int OFF_REC = OFF_Y + 65536;                  // record halves of the second token half
    static constexpr int OFF_PREF = OFF_REC + NT * 4;              // tile prefix per episode, counts
    static constexpr int OFF_BAR = ((OFF_PREF + (2 * MAXB + 1) * 4 + 7) / 8) * 8;
    static constexpr int TOTAL = OFF_BAR + 256 + 1024;             // + slack for the 1024-byte alignment
    static_assert(TOTAL <= 232448, "the streaming kernel's buffers exceed the 227 KB a CTA may use");
    static constexpr int TMEM_COLS = NTOK == 64 ? 256 : 128;       // D1 + two D2 slots, power of two
};

#define wait_bar(bar, parity) wait_bar_at((bar), (parity), __LINE__)

#ifdef RM_PHASE_TIMING
__device__ long long g_st_stamps[64];
__device__ __forceinline__ long long st_now() {
    long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define RM_ST(i) do { if (blockIdx.x == 0 && k == 0) g_st_stamps[(i)] = st_now(); } while (0)
#else
#define RM_ST(i) do { } while (0)
#endif

constexpr int SE = 288;                // threads: 4 epilogue warps (0-3), 4 loader warps (4-7), issuer warp (8)

// GATHER: the tile's neurons come from an index list, their rows are gathered with 16-byte cp.async (about 16 bytes
// per clock and SM, the limit of this kernel on lists).  Otherwise the tile is 64 consecutive rows of the layer (dense
// passes, compact layers) and a whole 64 x 64 block arrives as one tensor-map box.  x always arrives as one box.
template <int NTOK, bool EQ4, bool GATHER>
__global__ void __launch_bounds__(SE, 1) stream_tile_kernel(const StreamArgs a, const __grid_constant__ CUtensorMap tmW,
                                                            const __grid_constant__ CUtensorMap tmX,
                                                            const __grid_constant__ CUtensorMap tmOut,
                                                            const __grid_constant__ CUtensorMap tmYa) {
    using S = SmemST<NTOK>;
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* gbase = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t sRing = base + S::OFF_RING, sHT = base + S::OFF_HT;
    float* gY = reinterpret_cast<float*>(gbase + S::OFF_Y);
    float* gRec = reinterpret_cast<float*>(gbase + S::OFF_REC);
    int* gPref = reinterpret_cast<int*>(gbase + S::OFF_PREF);
    int* gCnt = gPref + MAXB + 1;
    const uint32_t bar0 = base + S::OFF_BAR;
    auto full = [&](int s) { return bar0 + 8 * s; };               // a stage's boxes have landed
    auto empty = [&](int s) { return bar0 + 48 + 8 * s; };         // the products reading a stage are complete
    const uint32_t d1_full = bar0 + 96, d1_free = bar0 + 104, h_full = bar0 + 112, h_free = bar0 + 120;
    auto d2_full = [&](int s) { return bar0 + 128 + 8 * s; };
    auto d2_free = [&](int s) { return bar0 + 144 + 8 * s; };
    const uint32_t s_tmem = bar0 + 160;
    volatile uint32_t* g_tmem = reinterpret_cast<volatile uint32_t*>(gbase + S::OFF_BAR + 160);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int H = a.H, T = a.T, Hs = H / 8;
    const int KBN = H / 64, MBN = H / 128;                         // stages per tile: gate/up blocks, down blocks
    const int anchor_mode = EQ4 ? a.anchor_mode : (int)RM_ANCHOR_NONE;
    const float* const gate = EQ4 ? a.gate : nullptr;

    if (tid == 0) {
        for (int s = 0; s < NSTAGE; ++s) { mbar_init(full(s), GATHER ? 129 : 1); mbar_init(empty(s), 1); }
        mbar_init(d1_full, 1); mbar_init(d1_free, 128); mbar_init(h_full, 128); mbar_init(h_free, 1);
        for (int s = 0; s < 2; ++s) { mbar_init(d2_full(s), 1); mbar_init(d2_free(s), 128); }
        fence_mbar_init();
        int acc = 0;
        const int cap = (int)(a.list_cap < (int64_t)a.I ? a.list_cap : (int64_t)a.I);
        for (int b = 0; b < a.B; ++b) {
            int c = a.I;
            if (a.count) {
                c = a.count[(size_t)b * a.count_stride];
                if (c < 0 || c > cap) { rm_set_status(a.status, RM_ERR_INDEX); c = c < 0 ? 0 : cap; }
            }
            gCnt[b] = c;
            gPref[b] = acc;
            acc += (c + NT - 1) / NT;
        }
        gPref[a.B] = acc;
    }
    if (warp == 8) tmem_alloc(s_tmem, S::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d1 = *g_tmem;
    pdl_launch_dependents();

    const int tiles_total = gPref[a.B];
    bool gave_up = false;
    auto wait_bar_at = [&](uint32_t bar, uint32_t parity, int line) {
        if (!mbar_wait(bar, parity)) {
            rm_set_status_at(a.status, RM_ERR_TIMEOUT, (line << 12) | (int)(blockIdx.x & 0xfffu));
            gave_up = true;
        }
    };
    auto episode_of = [&](int g) {
        int b = 0;
        while (gPref[b + 1] <= g) ++b;
        return b;
    };
    // neuron of slot q of tile g (-1: past the end of the list, or an index outside the layer)
    auto neuron_of = [&](int g, int b, int q, bool report) {
        const int p0 = (g - gPref[b]) * NT;
        int n = -1;
        if (p0 + q < gCnt[b]) {
            n = a.idx ? __ldg(a.idx + (size_t)b * a.idx_stride + p0 + q) : p0 + q;
            if (n < 0 || n >= a.I) {
                if (report) rm_set_status(a.status, RM_ERR_INDEX);
                n = -1;
            }
        }
        return n;
    };

    constexpr uint32_t IDESC_GU = idesc_bf16_f32(128, NTOK, false, false);
    constexpr uint32_t IDESC_DN = idesc_bf16_f32(128, NTOK, true, true);
    const uint64_t desc_k = smem_desc_sw128(0, 16, 1024);
    const uint64_t desc_mn = smem_desc_sw128(0, 8192, 1024);
    constexpr uint32_t GU_TX = W_BYTES + NTOK * 128, DN_TX = W_BYTES;

    if (warp >= 4 && warp < 8) {
        // ================================================================ loaders
        const int lt = tid - 128;                                  // loader thread 0..127
        const int r0 = lt >> 3, ch = lt & 7;                       // gathers: rows r0 + 16 i, 16-byte chunk ch
        uint32_t blk = 0;                                          // stages filled so far
        bool waited = false;                                       // griddepcontrol.wait done (x depends on it)
        auto stage_of = [&](uint32_t bk) { return sRing + (bk % NSTAGE) * STAGE; };
        auto acquire = [&](uint32_t bk) {
            if (bk >= NSTAGE) wait_bar(empty(bk % NSTAGE), ((bk / NSTAGE) - 1) & 1);
        };
        for (int k = 0;; ++k) {
            const int g = (int)blockIdx.x + k * (int)gridDim.x;
            if (g >= tiles_total) break;
            const int b = episode_of(g);
            const int p0 = (g - gPref[b]) * NT;
            int nq[4];
            const __nv_bfloat16* row[4];
            if (GATHER) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    nq[i] = neuron_of(g, b, r0 + 16 * i, ch == 0);
                    row[i] = a.packed + (size_t)(nq[i] < 0 ? 0 : nq[i]) * 3 * H + ch * 8;
                }
            }
            if (lt == 0) RM_ST(0);
            // gate rows q and up rows 64 + q of columns 64 kb .. (GATHER: this thread's 8 pieces; else two boxes)
            auto issue_w = [&](int kb, uint32_t bk) {
                const uint32_t st = stage_of(bk), fb = full(bk % NSTAGE);
                const int col = kb * 64, j = col / Hs, x0 = j * 3 * Hs + (col - j * Hs);
                if (GATHER) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int q = r0 + 16 * i;
                        const uint32_t d = st + q * 128 + ((ch ^ (q & 7)) << 4);
                        cp_async16(d, row[i] + x0, nq[i] >= 0);
                        cp_async16(d + 64 * 128, row[i] + x0 + Hs, nq[i] >= 0);
                    }
                    if (lt == 0) mbar_arrive_expect_tx(fb, NTOK * 128);
                } else if (lt == 0) {
                    mbar_arrive_expect_tx(fb, GU_TX);
                    tma_load_2d(st, &tmW, x0, p0, fb);
                    tma_load_2d(st + 8192, &tmW, x0 + Hs, p0, fb);
                }
            };
            auto issue_x = [&](int kb, uint32_t bk) {
                if (lt == 0) tma_load_2d(stage_of(bk) + W_BYTES, &tmX, kb * 64, b * T, full(bk % NSTAGE));
                if (GATHER) cp_async_arrive_noinc(full(bk % NSTAGE));
            };
            int kb = 0;
            if (!waited) {
                // the weights do not depend on the previous kernel: fill the ring with them, then wait, then add x
                const int pre = KBN < NSTAGE ? KBN : NSTAGE;
                for (int i = 0; i < pre; ++i) issue_w(i, blk + i);
                pdl_wait();
                waited = true;
                if (lt == 0) RM_ST(1);
                for (int i = 0; i < pre; ++i) issue_x(i, blk + i);
                blk += pre;
                kb = pre;
            }
            for (; kb < KBN; ++kb, ++blk) {
                acquire(blk);
                issue_w(kb, blk);
                issue_x(kb, blk);
            }
            if (lt == 0) RM_ST(2);                                 // all gate/up blocks issued
            for (int mb = 0; mb < MBN; ++mb, ++blk) {              // down rows: 64 neurons x 128 output columns
                acquire(blk);
                const uint32_t st = stage_of(blk), fb = full(blk % NSTAGE);
                if (!GATHER && lt == 0) mbar_arrive_expect_tx(fb, DN_TX);
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
                    const int col = mb * 128 + cb * 64, j = col / Hs, x0 = j * 3 * Hs + 2 * Hs + (col - j * Hs);
                    if (GATHER) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int q = r0 + 16 * i;
                            cp_async16(st + cb * 8192 + q * 128 + ((ch ^ (q & 7)) << 4), row[i] + x0, nq[i] >= 0);
                        }
                    } else if (lt == 0) {
                        tma_load_2d(st + cb * 8192, &tmW, x0, p0, fb);
                    }
                }
                if (GATHER) {
                    if (lt == 0) mbar_arrive(fb);                  // the arrival that carries the x bytes in gate/up stages
                    cp_async_arrive_noinc(fb);
                }
            }
        }
        if (!waited) pdl_wait();
    } else if (warp < 4) {
        // ================================================================ epilogue: tensor memory -> h, output
        const int m = tid, w4 = warp;                              // accumulator lane of this thread
        const int q = m & 63, half = m >> 6;                       // its neuron slot; token half it finishes
        constexpr int TH = NTOK / 2;                               // tokens per half
        uint32_t mbc = 0;                                          // down blocks consumed so far
        for (int k = 0;; ++k) {
            const int g = (int)blockIdx.x + k * (int)gridDim.x;
            if (g >= tiles_total) break;
            const int b = episode_of(g);
            const int n = neuron_of(g, b, q, false);
            wait_bar(d1_full, k & 1);
            tc_fence_after();
            if (m == 0) RM_ST(8);
            float v[NTOK];
#pragma unroll
            for (int c0 = 0; c0 < NTOK; c0 += 32)
                tmem_ld32(tmem_d1 + ((uint32_t)(w4 * 32) << 16) + c0, *reinterpret_cast<float(*)[32]>(v + c0));
            tc_fence_before();
            mbar_arrive(d1_free);
            if (m == 0) RM_ST(40);
            // lanes 0..63 hold the gate rows, lanes 64..127 the up rows.  Thread (q, half 0) finishes tokens 0..TH-1
            // of neuron q, thread (q, half 1) tokens TH..NTOK-1: each passes the other the half it does not need.
            float* xg = gY;                                        // gate values of the second token half [t][q]
            float* xu = gY + TH * NT;                              // up values of the first token half   [t][q]
            if (half == 0) {
#pragma unroll
                for (int t = 0; t < TH; ++t) xg[t * NT + q] = v[TH + t];
            } else {
#pragma unroll
                for (int t = 0; t < TH; ++t) xu[t * NT + q] = v[t];
            }
            named_barrier(1, 128);
            if (m == 0) RM_ST(41);
            const int tb = half * TH;                              // first token of this thread
            float hv[TH];
            float rec = 0.f;
            // in stages over all TH elements, so that the exponentials and divisions of different tokens overlap (one
            // warp per scheduler runs this: a token-by-token chain costs ~140 clocks per token)
            {
                float e[TH];
#pragma unroll
                for (int t = 0; t < TH; ++t) {
                    const float gg = half == 0 ? v[t] : xg[t * NT + q];
                    hv[t] = gg;
                    e[t] = __expf(-1.5957691216057308f * (gg + 0.044715f * gg * gg * gg));
                }
#pragma unroll
                for (int t = 0; t < TH; ++t) e[t] = __fdividef(hv[t], 1.0f + e[t]);     // GeLU-tanh(g) = g / (1 + exp(-2z))
#pragma unroll
                for (int t = 0; t < TH; ++t) {
                    const float uu = half == 0 ? xu[t * NT + q] : v[TH + t];
                    hv[t] = (tb + t < T && n >= 0) ? e[t] * uu : 0.f;
                    rec += fabsf(hv[t]);
                }
            }
            if (anchor_mode != RM_ANCHOR_NONE && n >= 0) {
                float* hap = a.h_anchor + ((size_t)b * a.I + n) * a.h_stride + tb;
                if (anchor_mode == RM_ANCHOR_WRITE) {
#pragma unroll
                    for (int t = 0; t < TH; t += 4)
                        if (tb + t < T) *reinterpret_cast<float4*>(hap + t) = make_float4(hv[t], hv[t + 1], hv[t + 2], hv[t + 3]);
                } else {
#pragma unroll
                    for (int t = 0; t < TH; t += 4)
                        if (tb + t < T) {
                            const float4 f = *reinterpret_cast<const float4*>(hap + t);
                            hv[t] -= f.x;
                            if (tb + t + 1 < T) hv[t + 1] -= f.y;
                            if (tb + t + 2 < T) hv[t + 2] -= f.z;
                            if (tb + t + 3 < T) hv[t + 3] -= f.w;
                        }
                }
            }
            if (a.record) {
                if (half == 1) gRec[q] = rec;
                named_barrier(1, 128);
                if (half == 0 && n >= 0) {
                    rec += gRec[q];
                    a.record[(size_t)b * a.record_stride + n] = a.record_scale ? rec * a.record_scale[n] : rec;
                }
            }
            if (m == 0) RM_ST(42);
            if (k > 0) wait_bar(h_free, (k - 1) & 1);              // the previous tile's down products are complete
            // row q of the h tile: 64 tokens in bf16, 16-byte chunks swizzled by the row; hi at 0, lo at 8 KB
            {
                unsigned char* rowp = gbase + S::OFF_HT + q * 128;
#pragma unroll
                for (int c = 0; c < TH / 8; ++c) {
                    uint32_t hi[4], lo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float f0 = hv[c * 8 + 2 * e], f1 = hv[c * 8 + 2 * e + 1];
                        const __nv_bfloat162 h2 = __floats2bfloat162_rn(f0, f1);
                        const float2 hf = __bfloat1622float2(h2);
                        const __nv_bfloat162 l2 = __floats2bfloat162_rn(f0 - hf.x, f1 - hf.y);
                        hi[e] = *reinterpret_cast<const uint32_t*>(&h2);
                        lo[e] = *reinterpret_cast<const uint32_t*>(&l2);
                    }
                    const int off = (((tb >> 3) + c) ^ (q & 7)) << 4;
                    *reinterpret_cast<uint4*>(rowp + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<uint4*>(rowp + NT * 128 + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(h_full);
            if (m == 0) RM_ST(9);
            // finished down blocks: lane = output column, token columns.  Transposed through shared memory into
            // [token][128 columns]; the copy engine adds the block to the output as one box of the [B, T, H] tensor
            // map (rows past T fall outside the map and are dropped).  The two staging buffers alternate, so one is
            // read while the other fills; the anchor step fills both per block, the ungated block for y_anchor and
            // the gated one for the output.
            const bool ya_b = anchor_mode == RM_ANCHOR_WRITE;
            for (int mb = 0; mb < MBN; ++mb, ++mbc) {
                const int slot = mbc & 1;
                wait_bar(d2_full(slot), (mbc >> 1) & 1);
                tc_fence_after();
                if (m == 0) RM_ST(10 + mb);
                float y[NTOK];
#pragma unroll
                for (int c0 = 0; c0 < NTOK; c0 += 32)
                    tmem_ld32(tmem_d1 + NTOK * (1 + slot) + ((uint32_t)(w4 * 32) << 16) + c0,
                              *reinterpret_cast<float(*)[32]>(y + c0));
                tc_fence_before();
                mbar_arrive(d2_free(slot));
                if (m == 0) {                                      // the box(es) sent from the buffer(s) about to be filled have left
                    if (ya_b) bulk_wait_read_all();
                    else bulk_wait_read_but_one();
                }
                named_barrier(1, 128);                             // the previous block's rows have been read
                if (!ya_b) {
                    float* gYb = gY + (mbc & 1) * 8192;            // the copy engine reads one buffer while the other fills
                    const float gm = gate ? gate[(size_t)b * H + mb * 128 + m] : 1.f;
#pragma unroll
                    for (int t = 0; t < NTOK; ++t)
                        if (t < T) gYb[t * 128 + m] = gm * y[t];
                    fence_proxy_async_smem();
                    named_barrier(1, 128);
                    if (m == 0) {
                        tensor_reduce_add_3d(&tmOut, mb * 128, 0, b, smem_u32(gYb));
                        bulk_commit();
                    }
                } else {
                    const float gm = gate ? gate[(size_t)b * H + mb * 128 + m] : 1.f;
#pragma unroll
                    for (int t = 0; t < NTOK; ++t)
                        if (t < T) {
                            gY[t * 128 + m] = y[t];
                            gY[8192 + t * 128 + m] = gm * y[t];
                        }
                    fence_proxy_async_smem();
                    named_barrier(1, 128);
                    if (m == 0) {
                        tensor_reduce_add_3d(&tmYa, mb * 128, 0, b, smem_u32(gY));
                        tensor_reduce_add_3d(&tmOut, mb * 128, 0, b, smem_u32(gY + 8192));
                        bulk_commit();
                    }
                }
                if (m == 0) RM_ST(30 + mb);
            }
            if (m == 0) bulk_wait_read_all();
            named_barrier(1, 128);                                 // the exchange area is free for the next tile
        }
    } else if (warp == 8) {
        // ================================================================ issuer: the whole warp runs the loop and one
        // elected lane issues (a loop that only lane 0 runs costs 100-150 clocks more per stage, and the tensor pipe
        // idles while the issuing thread does anything else).  The test of the next stage's barrier (~200 clocks even
        // when the data is there) is started behind the products of the current stage, so that it runs while they do.
        uint32_t blk = 0, mbc = 0;
        bool next_ok = false;                                      // the stage about to be used is known to have landed
        auto stage_ready = [&]() {
            if (!next_ok) wait_bar(full(blk % NSTAGE), (blk / NSTAGE) & 1);
        };
        auto look_ahead = [&]() {
            next_ok = __all_sync(0xffffffffu, mbar_test_wait(full((blk + 1) % NSTAGE), ((blk + 1) / NSTAGE) & 1));
        };
        for (int k = 0;; ++k) {
            const int g = (int)blockIdx.x + k * (int)gridDim.x;
            if (g >= tiles_total) break;
            if (k > 0) wait_bar(d1_free, (k - 1) & 1);             // the epilogue has read the previous D1
            tc_fence_after();
            for (int kb = 0; kb < KBN; ++kb, ++blk) {
                const uint32_t st = sRing + (blk % NSTAGE) * STAGE;
                stage_ready();
                if (lane == 0) {
                    if (kb == 0) RM_ST(3);
                    if (kb == KBN - 1) RM_ST(4);
                }
                if (GATHER) fence_proxy_async_smem();
                tc_fence_after();
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        mma_bf16_ss(tmem_d1, desc_k | desc_addr(st + ks * 32), desc_k | desc_addr(st + W_BYTES + ks * 32),
                                    IDESC_GU, (kb | ks) != 0);
                    mma_commit(empty(blk % NSTAGE));
                }
                __syncwarp();
                look_ahead();
            }
            if (elect_one()) mma_commit(d1_full);
            __syncwarp();
            if (lane == 0) RM_ST(5);
            wait_bar(h_full, k & 1);
            if (lane == 0) RM_ST(6);
            for (int mb = 0; mb < MBN; ++mb, ++blk, ++mbc) {
                const int slot = mbc & 1;
                const uint32_t st = sRing + (blk % NSTAGE) * STAGE;
                if (mbc >= 2) wait_bar(d2_free(slot), ((mbc >> 1) - 1) & 1);
                stage_ready();
                if (GATHER) fence_proxy_async_smem();
                tc_fence_after();
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const uint64_t aa = desc_mn | desc_addr(st + ks * 2048);
                        mma_bf16_ss(tmem_d1 + NTOK * (1 + slot), aa, desc_mn | desc_addr(sHT + ks * 2048), IDESC_DN, ks != 0);
                        mma_bf16_ss(tmem_d1 + NTOK * (1 + slot), aa, desc_mn | desc_addr(sHT + NT * 128 + ks * 2048), IDESC_DN, true);
                    }
                    mma_commit(empty(blk % NSTAGE));
                    mma_commit(d2_full(slot));
                }
                __syncwarp();
                look_ahead();
            }
            if (elect_one()) mma_commit(h_free);
            __syncwarp();
            if (lane == 0) RM_ST(7);
        }
    }
    tc_fence_before();
    if (__syncthreads_or(gave_up)) linger_after_timeout();
    if (warp == 8) tmem_dealloc(tmem_d1, S::TMEM_COLS);
}

// ---- tensor maps (host).  cuTensorMapEncodeTiled is taken from the driver through the runtime, so the library does
// not link against libcuda.
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

// bf16 matrix [rows, cols] row-major, boxes of box_rows x 64 columns (128 bytes), 128-byte swizzle
int make_map(CUtensorMap* tm, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return RM_ERR_UNSUPPORTED;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * sizeof(__nv_bfloat16)};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t es[2] = {1, 1};
    const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? RM_OK : RM_ERR_CUDA;
}

// fp32 output [B, T, H] as a 3-d map, boxes of box_rows token rows x 128 columns of one episode, no swizzle: token rows
// past T lie outside the map, so a box that covers them neither reads nor adds them
int make_map_out(CUtensorMap* tm, const float* ptr, uint64_t B, uint64_t T, uint64_t H, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return RM_ERR_UNSUPPORTED;
    cuuint64_t dims[3] = {H, T, B};
    cuuint64_t strides[2] = {H * sizeof(float), T * H * sizeof(float)};
    cuuint32_t box[3] = {128, box_rows, 1};
    cuuint32_t es[3] = {1, 1, 1};
    const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(ptr), dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? RM_OK : RM_ERR_CUDA;
}

template <int NTOK>
int launch_tiles(rm_ctx* ctx, const StreamArgs& a, int n_ctas, cudaStream_t s) {
    using S = SmemST<NTOK>;
    const bool eq4 = a.anchor_mode != RM_ANCHOR_NONE || a.gate != nullptr;
    const bool gather = a.idx != nullptr;
    auto kern = gather ? (eq4 ? stream_tile_kernel<NTOK, true, true> : stream_tile_kernel<NTOK, false, true>)
                       : (eq4 ? stream_tile_kernel<NTOK, true, false> : stream_tile_kernel<NTOK, false, false>);
    static rm_smem_configured configured = {};
    if (!configured.covers(ctx->device, S::TOTAL)) {
        RM_CUDA_TRY(cudaFuncSetAttribute(stream_tile_kernel<NTOK, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::TOTAL));
        RM_CUDA_TRY(cudaFuncSetAttribute(stream_tile_kernel<NTOK, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::TOTAL));
        RM_CUDA_TRY(cudaFuncSetAttribute(stream_tile_kernel<NTOK, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::TOTAL));
        RM_CUDA_TRY(cudaFuncSetAttribute(stream_tile_kernel<NTOK, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::TOTAL));
        configured.set(ctx->device, S::TOTAL);
    }
    CUtensorMap tmW, tmX, tmOut, tmYa;
    int rc = make_map(&tmW, a.packed, (uint64_t)a.I, (uint64_t)3 * a.H, NT);       // used without a list only
    if (rc != RM_OK) return rc;
    rc = make_map(&tmX, a.x, (uint64_t)a.B * a.T, (uint64_t)a.H, NTOK);
    if (rc != RM_OK) return rc;
    rc = make_map_out(&tmOut, a.r_out, (uint64_t)a.B, (uint64_t)a.T, (uint64_t)a.H, NTOK);
    if (rc != RM_OK) return rc;
    // the anchor step's second target; any valid map otherwise (not used)
    rc = make_map_out(&tmYa, a.anchor_mode == RM_ANCHOR_WRITE ? a.y_anchor : a.r_out, (uint64_t)a.B, (uint64_t)a.T,
                      (uint64_t)a.H, NTOK);
    if (rc != RM_OK) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_ctas);
    cfg.blockDim = dim3(SE);
    cfg.dynamicSmemBytes = S::TOTAL;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, a, tmW, tmX, tmOut, tmYa));
    ctx->launches++;
    return RM_OK;
}

}  // namespace

int rm_make_out_map(void* tensor_map, const float* ptr, int B, int T, int H, int box_rows) {
    return make_map_out(static_cast<CUtensorMap*>(tensor_map), ptr, (uint64_t)B, (uint64_t)T, (uint64_t)H, (uint32_t)box_rows);
}

int rm_stream_debug_stamps(long long* host_out) {
#ifdef RM_PHASE_TIMING
    return cudaMemcpyFromSymbol(host_out, g_st_stamps, sizeof(long long) * 64) == cudaSuccess ? RM_OK : RM_ERR_CUDA;
#else
    (void)host_out;
    return RM_ERR_UNSUPPORTED;
#endif
}

bool rm_stream_supported(const rm_ctx* ctx, int B, int T) {
    return (ctx->g.H == 1024 || ctx->g.H == 2048) && T >= 1 && T <= 64 && B >= 1 && B <= MAXB && ctx->sm_count > 0;
}

// One layer.  Without la.x: la.r_in is normalised into x_scratch and la.r_out (a different buffer) is set to the
// residual (+ gate * y_anchor in update steps) before the tiles are added.  With la.x the caller has prepared la.r_out.
int rm_launch_layer_stream(rm_ctx* ctx, const rm_layer_args& la, __nv_bfloat16* x_scratch, bool pdl, cudaStream_t s) {
    const rm_geom& g = ctx->g;
    const __nv_bfloat16* x = la.x;
    if (!x) {
        PrepArgs p{};
        p.r_in = la.r_in;
        p.x = x_scratch;
        p.r_out = la.r_out;
        p.y_anchor = la.anchor_mode == RM_ANCHOR_UPDATE ? la.y_anchor : nullptr;
        p.gate = la.gate;
        p.T = la.T;
        p.H = g.H;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(la.B * la.T);
        cfg.blockDim = dim3(256);
        cfg.stream = s;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at;
        cfg.numAttrs = pdl ? 1 : 0;
        RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, stream_prep_kernel, p));
        ctx->launches++;
        x = x_scratch;
    }
    StreamArgs a{};
    a.packed = la.packed;
    a.x = x;
    a.r_out = la.r_out;
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
    a.H = g.H;
    a.I = g.I;
    a.status = ctx->d_status;
    a.anchor_mode = la.anchor_mode;
    a.y_anchor = la.y_anchor;
    a.h_anchor = la.h_anchor;
    a.h_stride = la.h_stride;
    a.gate = la.gate;
    const int per_episode = la.count ? rm_effective_count_hint(ctx) : g.I;
    long long tiles = per_episode > 0 ? (long long)((per_episode + NT - 1) / NT) * la.B : 0;
    int n_ctas = ctx->sm_count;
    if (tiles > 0 && tiles < n_ctas) n_ctas = (int)tiles;
    if (ctx->max_clusters_override > 0 && ctx->max_clusters_override < n_ctas) n_ctas = ctx->max_clusters_override;
    return la.T <= 32 ? launch_tiles<32>(ctx, a, n_ctas, s) : launch_tiles<64>(ctx, a, n_ctas, s);
}
