// Whole-step kernel of the masked gated MLP stack: ONE launch runs every layer of a denoising step.
//
// The mask of every layer is known before the step starts (it comes from an earlier, similar execution), so every
// weight address of the step is known too: loader warps stream the step's weight rows through a shared-memory ring
// without ever waiting for a layer boundary, and only the arithmetic follows the layer-to-layer dependency.
//
// Grid: clusters of 8 CTAs, all co-resident (one CTA per SM).  Per layer and episode (an "item") the active list is
// cut evenly over the clusters; a cluster walks its run in tiles of up to 256 neurons.  Inside a tile
//   gate/up : CTA j takes up to 32 of the tile's neurons and computes their gate and up rows against the whole
//             width H -- A = the neurons' weight rows (64 rows: gate and up interleaved, K-major, 128-byte swizzle,
//             gathered by 16-byte cp.async), B = x (64 token rows, one tensor-map box per 64 columns),
//             D1[64 x 64] in tensor memory.  No partial sums cross CTAs.
//   GLU     : h = gelu_tanh(g) * u from tensor memory, split into a bf16 pair hi + lo, written to this CTA's h tile
//             and copied to the 7 peers' h tiles (bulk copies counted on the receivers' mbarriers).
//   down    : CTA j owns output columns [j H/8, (j+1) H/8): D2[H/8 x (hi | lo tokens)] += Wd-slice * h over ALL the
//             tile's neurons, accumulated in tensor memory over the item's tiles.
// At the end of an item the CTA adds its [T x H/8] partial to the fp32 residual stream with red.global.add and
// arrives on the episode's counter.  The next layer's input is prepared per cluster: once the counter shows that
// every CTA has added its part, the cluster's CTAs normalise the token rows (x = bf16(r rsqrt(mean r^2 + 1e-6)))
// into the cluster's own copy of x in global memory, tell one another through remote mbarrier arrivals, and
// stream x from there.
//
// Every wait is bounded; a wait that runs out records RM_ERR_TIMEOUT (with its source line), raises the launch's
// abort flag, and every role leaves its loop at the next check.  CTAs leave together (cluster barrier at the end).
#include <cuda.h>

#include <mutex>

#include "rm_common.cuh"
#include "rm_sm100.cuh"

using namespace sm100;

namespace {

constexpr int CS = 8;                  // CTAs per cluster = column slices of the packed layout
constexpr int NT = 32;                 // neurons whose gate/up rows one CTA computes per tile
constexpr int CT = CS * NT;            // slots of a cluster tile
constexpr int NTOK = 64;               // token rows (padded)
constexpr int XS = 4;                  // x ring: stages of one 64-column box (8 KB)
constexpr int X_BYTES = NTOK * 128;
constexpr int W_RING = 96 * 1024;      // weight ring
constexpr int H_HALF = CT * 128;       // h tile: hi block, then lo block (each 256 slots x 64 tokens bf16)
constexpr int MAXL = 64, MAXB = 16;
constexpr int NTHREADS = 576;          // warps: 0-7 epilogue, 8-11 loaders, 12-15 normalisation, 16 issuer, 17 x boxes
constexpr int W_LOAD0 = 8, W_NORM0 = 12, W_MMA = 16, W_XTMA = 17;
constexpr int SYNC_ABORT = MAXB;       // sync[0..MAXB): per-episode arrival counters; sync[MAXB]: abort flag

struct PArgs {
    const __nv_bfloat16* packed[MAXL];
    float* r;                          // [B,T,H] fp32: holds r_0 on entry and r_L on exit (layers add in place)
    __nv_bfloat16* xbuf;               // [clusters][2][64][H] bf16: the clusters' own copies of x
    const int32_t* idx;                // list (b, l) at idx + b * idx_b_stride + l * idx_l_stride; NULL: positions
    const int32_t* count;              // count (b, l) at count[b * count_b_stride + l]; NULL: every neuron
    int64_t idx_b_stride, idx_l_stride, list_cap, count_b_stride;
    float* record;                     // record (b, l, n) at record[b * rec_b_stride + l * I + n]; NULL: none
    int64_t rec_b_stride;
    const float* record_scale;         // [L, I] or NULL
    int* sync;
    int* status;
    int L, B, T, I;
    int x_ext;                         // layer 0 takes x from the caller's buffer (single-layer entry): no normalisation
};

#ifdef RM_PHASE_TIMING
__device__ long long g_ps_stamps[64 * 128 * 16];
__device__ __forceinline__ long long ps_now() {
    long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define RM_PS(item, slot) do { if ((item) < 64 && blockIdx.x < 128) g_ps_stamps[((item) * 128 + blockIdx.x) * 16 + (slot)] = ps_now(); } while (0)
#else
#define RM_PS(item, slot) do { } while (0)
#endif

__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_gpu(int* p, int v) {
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// arrive on the mbarrier at the same shared-memory offset in every CTA of `mask` once all MMAs issued so far by
// this thread have completed
__device__ __forceinline__ void mma_commit_mc(uint32_t bar, uint16_t mask) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
// OR of a predicate over the threads of a named barrier: one decision for the whole group
__device__ __forceinline__ bool named_barrier_or(int id, int count, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "barrier.cta.red.or.pred q, %2, %3, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"((uint32_t)pred), "r"(id), "r"(count) : "memory");
    return r != 0;
}

// ---- the split of an item over clusters, tiles and CTAs (every role computes it the same way)
struct Run { int start, n, ntiles; };
__device__ __forceinline__ Run cluster_run(int K, int c, int NC) {
    Run r;
    r.start = (int)((long long)K * c / NC);
    r.n = (int)((long long)K * (c + 1) / NC) - r.start;
    r.ntiles = (r.n + CT - 1) / CT;
    return r;
}
__device__ __forceinline__ void tile_span(const Run& r, int i, int& t0, int& ts) {
    const int a = (int)((long long)r.n * i / r.ntiles), b = (int)((long long)r.n * (i + 1) / r.ntiles);
    t0 = r.start + a;
    ts = b - a;                                                    // <= 256
}
__device__ __forceinline__ void cta_span(int ts, int j, int& off, int& nj) {
    off = ts * j / CS;
    nj = ts * (j + 1) / CS - off;                                  // <= 32
}

// Cursor over the tiles this cluster walks during the step, in order.
struct Cur {
    int item, l, b, i;
    Run run;
    int seq;                           // tiles before this one
    int ni;                            // non-empty items before this one
    int use;                           // uses of the cluster's x buffer before this item
    bool valid;
};
struct Env { const int* sK; int L, B, c, NC, x_ext; };
__device__ __forceinline__ bool item_ext(const Env& e, int l) { return e.x_ext && l == 0; }
__device__ __forceinline__ void cur_seek(Cur& k, const Env& e) {      // to the first non-empty item at or after k.item
    const int n_items = e.L * e.B;
    while (k.item < n_items) {
        k.l = k.item / e.B;
        k.b = k.item - k.l * e.B;
        k.run = cluster_run(e.sK[k.item], e.c, e.NC);
        if (k.run.ntiles > 0) { k.valid = true; k.i = 0; return; }
        ++k.item;
    }
    k.valid = false;
}
__device__ __forceinline__ void cur_init(Cur& k, const Env& e) {
    k.item = 0; k.seq = 0; k.ni = 0; k.use = 0; k.i = 0;
    cur_seek(k, e);
}
__device__ __forceinline__ void cur_next(Cur& k, const Env& e) {
    ++k.seq;
    if (++k.i < k.run.ntiles) return;
    if (!item_ext(e, k.l)) ++k.use;
    ++k.ni;
    ++k.item;
    cur_seek(k, e);
}

template <int HS8>
struct Geo {
    static constexpr int H = 8 * HS8;
    static constexpr int NSB = HS8 / 64;               // 64-column boxes per column slice
    static constexpr int NMB = HS8 / 128;              // 128-column output blocks per slice
    static constexpr int SB = HS8 * 128;               // bytes of a weight stage: 64 rows x HS8 columns
    static constexpr int NW = W_RING / SB;
    static constexpr int ND2 = NMB == 1 ? 2 : 1;       // down accumulators (an item's flush overlaps the next item's products)
    static constexpr int D2_COL = 2 * NTOK;            // tensor memory: D1[2] at 0 and 64, D2 from 128
    static constexpr int OFF_W = 0;
    static constexpr int OFF_X = OFF_W + W_RING;
    static constexpr int OFF_H = OFF_X + XS * X_BYTES;
    static constexpr int OFF_K = OFF_H + 2 * H_HALF;   // counts of the items
    static constexpr int OFF_REC = OFF_K + MAXL * MAXB * 4;
    static constexpr int OFF_BAR = OFF_REC + NT * 4;
    static constexpr int TOTAL = OFF_BAR + 512 + 1024; // + slack for the 1024-byte alignment
    static_assert(TOTAL <= 232448, "buffers exceed the shared memory of a CTA");
};

template <int HS8>
__global__ void __launch_bounds__(NTHREADS, 1) step_kernel(const __grid_constant__ PArgs a,
                                                          const __grid_constant__ CUtensorMap tmX,
                                                          const __grid_constant__ CUtensorMap tmXext) {
    using G = Geo<HS8>;
    constexpr int H = G::H, NSB = G::NSB, NMB = G::NMB, SB = G::SB, NW = G::NW, ND2 = G::ND2;
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* gbase = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t sW = base + G::OFF_W, sX = base + G::OFF_X, sH = base + G::OFF_H;
    int* sK = reinterpret_cast<int*>(gbase + G::OFF_K);
    float* sRec = reinterpret_cast<float*>(gbase + G::OFF_REC);
    const uint32_t bar0 = base + G::OFF_BAR;
    auto w_full = [&](int s) { return bar0 + 8 * s; };              // up to 6
    auto w_empty = [&](int s) { return bar0 + 48 + 8 * s; };
    auto x_full = [&](int s) { return bar0 + 96 + 8 * s; };         // 4
    auto x_empty = [&](int s) { return bar0 + 128 + 8 * s; };
    auto d1_full = [&](int s) { return bar0 + 160 + 8 * s; };       // 2
    auto d2_full = [&](int s) { return bar0 + 176 + 8 * s; };       // 2
    auto d2_empty = [&](int s) { return bar0 + 192 + 8 * s; };
    auto x_ready = [&](int s) { return bar0 + 208 + 8 * s; };       // 2
    auto x_free = [&](int s) { return bar0 + 224 + 8 * s; };
    const uint32_t h_full = bar0 + 240, h_free = bar0 + 248;
    const uint32_t s_tmem = bar0 + 256;
    volatile uint32_t* g_tmem = reinterpret_cast<volatile uint32_t*>(gbase + G::OFF_BAR + 256);
    volatile int* sAbort = reinterpret_cast<volatile int*>(gbase + G::OFF_BAR + 264);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int j = (int)cluster_ctarank(), c = (int)cluster_id_x(), NC = (int)cluster_count_x();
    const int T = a.T, L = a.L, B = a.B, I = a.I;
    const int n_ctas = (int)gridDim.x;
    const int n_items = L * B;

    if (tid == 0) {
        for (int s = 0; s < NW; ++s) { mbar_init(w_full(s), 128); mbar_init(w_empty(s), 1); }
        for (int s = 0; s < XS; ++s) { mbar_init(x_full(s), 1); mbar_init(x_empty(s), 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(d1_full(s), 1); mbar_init(d2_full(s), 1); mbar_init(d2_empty(s), 256);
            mbar_init(x_ready(s), CS); mbar_init(x_free(s), CS);
        }
        mbar_init(h_full, 1); mbar_init(h_free, CS);
        fence_mbar_init();
        *sAbort = 0;
    }
    {
        const int cap = (int)(a.list_cap < (int64_t)I ? a.list_cap : (int64_t)I);
        for (int it = tid; it < n_items; it += NTHREADS) {
            const int l = it / B, b = it - l * B;
            int k = I;
            if (a.count) {
                k = a.count[(size_t)b * a.count_b_stride + l];
                if (k < 0 || k > cap) { rm_set_status(a.status, RM_ERR_INDEX); k = k < 0 ? 0 : cap; }
            }
            sK[it] = k;
        }
    }
    if (warp == W_MMA) tmem_alloc(s_tmem, 512);
    if (warp >= W_NORM0 && warp < W_NORM0 + 4) {
        // token rows T..63 of the cluster's x copies stay zero for the whole step
        const int nw = warp - W_NORM0;
        for (int slot = 0; slot < 2; ++slot)
            for (int row = T + nw; row < NTOK; row += 4) {
                if ((row & 7) != j) continue;
                uint2* dst = reinterpret_cast<uint2*>(a.xbuf + ((size_t)(c * 2 + slot) * NTOK + row) * H);
                for (int e = lane; e < H / 4; e += 32) dst[e] = make_uint2(0u, 0u);
            }
        __threadfence();
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem = *g_tmem;
    Env env{sK, L, B, c, NC, a.x_ext};

    bool gave_up = false;
    auto timed_out = [&](int line) {
        rm_set_status_at(a.status, RM_ERR_TIMEOUT, (line << 12) | (int)(blockIdx.x & 0xfffu));
        gave_up = true;
        *sAbort = 1;
        atomicExch(a.sync + SYNC_ABORT, 1);
    };
    auto wait_at = [&](uint32_t bar, uint32_t parity, int line) {
        if (gave_up) return;
        for (uint32_t i = 0; i < (1u << 22); ++i) {
            if (mbar_try_wait(bar, parity)) return;
            if (i > 64) __nanosleep(32);
            if ((i & 1023u) == 1023u && (*sAbort || ((i & 16383u) == 16383u && ld_acquire_gpu(a.sync + SYNC_ABORT)))) {
                gave_up = true;
                *sAbort = 1;
                return;
            }
        }
        timed_out(line);
    };
#define WAIT(bar, parity) wait_at((bar), (parity), __LINE__)

    const uint64_t desc_k = smem_desc_sw128(0, 16, 1024);
    const uint64_t desc_mn_a = smem_desc_sw128(0, 8192, 1024);
    const uint64_t desc_mn_b = smem_desc_sw128(0, H_HALF, 1024);
    constexpr uint32_t IDESC_G = idesc_bf16_f32(64, NTOK, false, false);
    constexpr uint32_t IDESC_D = idesc_bf16_f32(128, 2 * NTOK, true, true);

    if (warp >= W_LOAD0 && warp < W_LOAD0 + 4) {
        // ================================================================ loaders: the step's weight rows, in the
        // order in which the issuer consumes them
        const int lt = tid - W_LOAD0 * 32, lw = lt >> 5;
        const int pc = lt & 7, r0 = lt >> 3;                       // gate/up: 16-byte piece, rows r0 + 16 q
        uint32_t wcnt = 0;
        auto acquire = [&]() {
            const int ws = wcnt % NW;
            if (wcnt >= (uint32_t)NW) WAIT(w_empty(ws), ((wcnt / NW) - 1) & 1);
            return sW + ws * SB;
        };
        auto list_of = [&](const Cur& k) {
            return a.idx ? a.idx + (size_t)k.b * a.idx_b_stride + (size_t)k.l * a.idx_l_stride : nullptr;
        };
        auto neuron = [&](const int32_t* list, int pos) {
            int n = list ? __ldg(list + pos) : pos;
            if (n < 0 || n >= I) { rm_set_status(a.status, RM_ERR_INDEX); n = -1; }
            return n;
        };
        auto load_g = [&](const Cur& k) {
            int t0, ts, off, nj;
            tile_span(k.run, k.i, t0, ts);
            cta_span(ts, j, off, nj);
            const int32_t* list = list_of(k);
            const __nv_bfloat16* src[4];
            bool ok[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = r0 + 16 * q, i = r >> 1;
                int n = -1;
                if (i < nj) n = neuron(list, t0 + off + i);
                ok[q] = n >= 0;
                src[q] = a.packed[k.l] + (size_t)(n < 0 ? 0 : n) * 3 * H + (r & 1) * HS8 + pc * 8;
            }
            for (int cc = 0; cc < CS; ++cc) {
                const uint32_t st = acquire();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int r = r0 + 16 * q;
                    const uint32_t d = st + (r >> 3) * 1024 + (r & 7) * 128 + ((pc ^ (r & 7)) << 4);
                    if (ok[q]) {
#pragma unroll
                        for (int sb = 0; sb < NSB; ++sb) cp_async16(d + sb * 8192, src[q] + cc * 3 * HS8 + sb * 64, true);
                    }
                }
                cp_async_arrive_noinc(w_full(wcnt % NW));
                ++wcnt;
            }
        };
        auto load_d = [&](const Cur& k) {
            int t0, ts;
            tile_span(k.run, k.i, t0, ts);
            const int32_t* list = list_of(k);
            const int kst = (ts + 15) >> 4, nst = (ts + 63) >> 6;
            constexpr int PPS = HS8 / 8;                           // 16-byte pieces of a neuron's down slice
            constexpr int SPW = 32 / PPS;                          // slots one warp instruction covers
            constexpr int NIT = 64 / (4 * SPW);
            const int piece = lane % PPS;
            for (int s = 0; s < nst; ++s) {
                const uint32_t st = acquire();
                int nn[NIT];
#pragma unroll
                for (int m = 0; m < NIT; ++m) {
                    const int slot = (lw + 4 * m) * SPW + lane / PPS, kk = 64 * s + slot;
                    nn[m] = kk < ts ? neuron(list, t0 + kk) : -1;
                }
#pragma unroll
                for (int m = 0; m < NIT; ++m) {
                    const int slot = (lw + 4 * m) * SPW + lane / PPS, kk = 64 * s + slot;
                    if (kk >= 16 * kst) continue;                  // beyond the last product step of the tile
                    const uint32_t d = st + (piece >> 3) * 8192 + slot * 128 + (((piece & 7) ^ (slot & 7)) << 4);
                    const __nv_bfloat16* p = a.packed[k.l] + (size_t)(nn[m] < 0 ? 0 : nn[m]) * 3 * H + j * 3 * HS8 + 2 * HS8 + piece * 8;
                    cp_async16(d, p, nn[m] >= 0);                  // unused slots of the last step: zeros
                }
                cp_async_arrive_noinc(w_full(wcnt % NW));
                ++wcnt;
            }
        };
        Cur g, d;
        cur_init(g, env);
        d = g;
        if (g.valid) { load_g(g); cur_next(g, env); }
        while (d.valid && !gave_up) {
            const bool ahead = g.valid && (g.item == d.item || B >= 2);
            if (ahead) { load_g(g); cur_next(g, env); }
            load_d(d);
            cur_next(d, env);
            if (!ahead && g.valid) { load_g(g); cur_next(g, env); }
        }
        cp_async_wait<0>();
    } else if (warp == W_XTMA) {
        // ================================================================ x boxes (one thread)
        if (lane == 0) {
            uint32_t xcnt = 0;
            Cur k;
            cur_init(k, env);
            int cur_item = -1;
            bool ext = false;
            int slot = 0;
            while (k.valid && !gave_up) {
                if (k.item != cur_item) {
                    cur_item = k.item;
                    ext = item_ext(env, k.l);
                    slot = k.use & 1;
                    if (!ext) {
                        const uint32_t ph = (k.use >> 1) & 1;
                        bool ok = false;
                        for (uint32_t i = 0; i < (1u << 22) && !ok; ++i) {
                            ok = mbar_try_wait_cluster(x_ready(slot), ph);
                            if (!ok && i > 64) __nanosleep(32);
                            if ((i & 1023u) == 1023u && *sAbort) break;
                        }
                        if (!ok) { if (!*sAbort) timed_out(__LINE__); gave_up = true; break; }
                        fence_proxy_async();
                        RM_PS(k.item, 0);
                    }
                }
                const int row = ext ? 0 : (c * 2 + slot) * NTOK;
                for (int cc = 0; cc < CS * NSB; ++cc) {
                    const int xs = xcnt % XS;
                    if (xcnt >= (uint32_t)XS) WAIT(x_empty(xs), ((xcnt / XS) - 1) & 1);
                    mbar_arrive_expect_tx(x_full(xs), X_BYTES);
                    tma_load_2d(sX + xs * X_BYTES, ext ? &tmXext : &tmX, cc * 64, row, x_full(xs));
                    ++xcnt;
                }
                cur_next(k, env);
            }
        }
    } else if (warp == W_MMA) {
        // ================================================================ issuer (one thread)
        if (lane == 0) {
            uint32_t wcnt = 0, xcnt = 0;
            auto issue_g = [&](const Cur& k) {
                const int buf = k.seq & 1;
                for (int cc = 0; cc < CS; ++cc) {
                    const int ws = wcnt % NW;
                    const uint32_t st = sW + ws * SB;
                    WAIT(w_full(ws), (wcnt / NW) & 1);
                    fence_proxy_async_smem();
#pragma unroll
                    for (int sb = 0; sb < NSB; ++sb) {
                        const int xs = xcnt % XS;
                        const uint32_t xt = sX + xs * X_BYTES;
                        WAIT(x_full(xs), (xcnt / XS) & 1);
                        if (cc == 0 && sb == 0 && k.i == 0) RM_PS(k.item, 1);
                        tc_fence_after();
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            mma_bf16_ss(tmem + buf * NTOK, desc_k | desc_addr(st + sb * 8192 + ks * 32),
                                        desc_k | desc_addr(xt + ks * 32), IDESC_G, (cc | sb | ks) != 0);
                        mma_commit(x_empty(xs));
                        ++xcnt;
                    }
                    mma_commit(w_empty(ws));
                    ++wcnt;
                }
                mma_commit(d1_full(buf));
                if (k.i == k.run.ntiles - 1 && !item_ext(env, k.l)) mma_commit_mc(x_free(k.use & 1), 0xff);
            };
            auto issue_d = [&](const Cur& k) {
                int t0, ts;
                tile_span(k.run, k.i, t0, ts);
                const int kst = (ts + 15) >> 4, nst = (ts + 63) >> 6;
                const int d2b = ND2 == 2 ? (k.ni & 1) : 0, nu = ND2 == 2 ? (k.ni >> 1) : k.ni;
                if (k.i == 0 && nu >= 1) WAIT(d2_empty(d2b), (nu - 1) & 1);
                WAIT(h_full, k.seq & 1);
                RM_PS(k.item, 4);
                tc_fence_after();
                const uint32_t d2 = tmem + G::D2_COL + d2b * (2 * NTOK);
                for (int s = 0; s < nst; ++s) {
                    const int ws = wcnt % NW;
                    const uint32_t st = sW + ws * SB;
                    WAIT(w_full(ws), (wcnt / NW) & 1);
                    fence_proxy_async_smem();
                    tc_fence_after();
                    const int nks = kst - 4 * s < 4 ? kst - 4 * s : 4;
                    for (int ks = 0; ks < nks; ++ks) {
                        const int kk = 4 * s + ks;
#pragma unroll
                        for (int mb = 0; mb < NMB; ++mb)
                            mma_bf16_ss(d2 + mb * (2 * NTOK), desc_mn_a | desc_addr(st + mb * 16384 + ks * 2048),
                                        desc_mn_b | desc_addr(sH + kk * 2048), IDESC_D, !(k.i == 0 && kk == 0));
                    }
                    mma_commit(w_empty(ws));
                    ++wcnt;
                }
                mma_commit_mc(h_free, 0xff);
                if (k.i == k.run.ntiles - 1) mma_commit(d2_full(d2b));
            };
            Cur g, d;
            cur_init(g, env);
            d = g;
            if (g.valid) { issue_g(g); cur_next(g, env); }
            while (d.valid && !gave_up) {
                const bool ahead = g.valid && (g.item == d.item || B >= 2);
                if (ahead) { issue_g(g); cur_next(g, env); }
                issue_d(d);
                cur_next(d, env);
                if (!ahead && g.valid) { issue_g(g); cur_next(g, env); }
            }
        }
    } else if (warp >= W_NORM0) {
        // ================================================================ normalisation: this cluster's copy of x
        const int nw = warp - W_NORM0;
        int use = 0;
        bool stop = false;
        for (int item = 0; item < n_items && !stop; ++item) {
            const int l = item / B, b = item - l * B;
            const Run run = cluster_run(sK[item], c, NC);
            if (run.ntiles == 0 || item_ext(env, l)) continue;
            const int slot = use & 1, nu = use >> 1;
            ++use;
            if (nu >= 1) WAIT(x_free(slot), (nu - 1) & 1);
            if (l > 0) {
                // every CTA has added its part of layer l-1 to this episode's rows
                const int target = n_ctas * l;
                if (lane == 0 && !gave_up) {
                    bool ok = false;
                    for (uint32_t i = 0; i < (1u << 21); ++i) {
                        if (ld_acquire_gpu(a.sync + b) >= target) { ok = true; break; }
                        if ((i & 255u) == 255u && (*sAbort || ld_acquire_gpu(a.sync + SYNC_ABORT))) break;
                    }
                    if (!ok) { if (!*sAbort && !ld_acquire_gpu(a.sync + SYNC_ABORT)) timed_out(__LINE__); gave_up = true; *sAbort = 1; }
                }
                __syncwarp();
            }
            if (nw == 0 && lane == 0) RM_PS(item, 8);
            const float* rb = a.r + (size_t)b * T * H;
            __nv_bfloat16* xb = a.xbuf + (size_t)(c * 2 + slot) * NTOK * H;
            for (int row = j + 8 * nw; row < T; row += 32) {
                const float4* src = reinterpret_cast<const float4*>(rb + (size_t)row * H);
                float4 v[H / 128];
                float ss = 0.f;
#pragma unroll
                for (int q = 0; q < H / 128; ++q) {
                    v[q] = __ldcg(src + lane + 32 * q);
                    ss = fmaf(v[q].x, v[q].x, ss); ss = fmaf(v[q].y, v[q].y, ss);
                    ss = fmaf(v[q].z, v[q].z, ss); ss = fmaf(v[q].w, v[q].w, ss);
                }
#pragma unroll
                for (int dd = 16; dd > 0; dd >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, dd);
                const float inv = 1.0f / sqrtf(ss / (float)H + 1e-6f);
                uint2* dst = reinterpret_cast<uint2*>(xb + (size_t)row * H);
#pragma unroll
                for (int q = 0; q < H / 128; ++q) {
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(v[q].x * inv, v[q].y * inv);
                    const __nv_bfloat162 hi = __floats2bfloat162_rn(v[q].z * inv, v[q].w * inv);
                    uint2 u;
                    u.x = *reinterpret_cast<const uint32_t*>(&lo);
                    u.y = *reinterpret_cast<const uint32_t*>(&hi);
                    dst[lane + 32 * q] = u;
                }
            }
            __threadfence();
            fence_proxy_async();
            stop = named_barrier_or(2, 128, gave_up || *sAbort);
            if (nw == 0 && lane < CS) mbar_arrive_remote(map_to_rank(x_ready(slot), lane));
            if (nw == 0 && lane == 0) RM_PS(item, 9);
        }
    } else {
        // ================================================================ epilogue (8 warps): GLU, h exchange, flush
        const int et = tid;                                         // 0..255
        const int q4 = warp & 3, ch = warp >> 2;                    // tensor-memory lane quarter; token half
        const bool act = lane < 16;                                 // rows of D1 (M = 64) sit in lanes 0..15 of a quarter
        const int ni_loc = 8 * q4 + (lane >> 1);                    // neuron of this lane among the CTA's 32
        const bool isup = lane & 1;
        int seq = 0, ni = 0;
        bool stop = false;
        for (int item = 0; item < n_items && !stop; ++item) {
            const int l = item / B, b = item - l * B;
            const Run run = cluster_run(sK[item], c, NC);
            const int32_t* list = a.idx ? a.idx + (size_t)b * a.idx_b_stride + (size_t)l * a.idx_l_stride : nullptr;
            for (int i = 0; i < run.ntiles && !stop; ++i, ++seq) {
                int t0, ts, off, nj;
                tile_span(run, i, t0, ts);
                cta_span(ts, j, off, nj);
                const int buf = seq & 1;
                int n = -1;
                if (act && ni_loc < nj) {
                    n = list ? __ldg(list + t0 + off + ni_loc) : t0 + off + ni_loc;
                    if (n < 0 || n >= I) n = -1;
                }
                WAIT(d1_full(buf), (seq >> 1) & 1);
                tc_fence_after();
                if (et == 0 && i == 0) RM_PS(item, 2);
                float v[32];
                tmem_ld32(tmem + buf * NTOK + ch * 32 + ((uint32_t)(q4 * 32) << 16), v);
                tc_fence_before();
                // lane pair (2m, 2m+1) holds the gate and the up row of one neuron for tokens 32 ch .. 32 ch + 31;
                // the even lane finishes the first 16 of them, the odd lane the last 16
                float hv[16];
                {
                    float gg[16], uu[16], e[16];
#pragma unroll
                    for (int r = 0; r < 16; ++r) {
                        const float mine = isup ? v[r] : v[16 + r];
                        const float got = __shfl_xor_sync(0xffffffffu, mine, 1);
                        gg[r] = isup ? got : v[r];
                        uu[r] = isup ? v[16 + r] : got;
                    }
#pragma unroll
                    for (int r = 0; r < 16; ++r) e[r] = __expf(-1.5957691216057308f * (gg[r] + 0.044715f * gg[r] * gg[r] * gg[r]));
#pragma unroll
                    for (int r = 0; r < 16; ++r) e[r] = __fdividef(gg[r], 1.0f + e[r]);
#pragma unroll
                    for (int r = 0; r < 16; ++r) hv[r] = n >= 0 ? e[r] * uu[r] : 0.f;
                }
                if (a.record) {
                    float rec = 0.f;
#pragma unroll
                    for (int r = 0; r < 16; ++r) rec += fabsf(hv[r]);
                    rec += __shfl_xor_sync(0xffffffffu, rec, 1);
                    if (ch == 1 && act && !isup) sRec[ni_loc] = rec;
                    named_barrier(1, 256);
                    if (ch == 0 && act && !isup && n >= 0) {
                        rec += sRec[ni_loc];
                        const float sc = a.record_scale ? a.record_scale[(size_t)l * I + n] : 1.f;
                        a.record[(size_t)b * a.rec_b_stride + (size_t)l * I + n] = a.record_scale ? rec * sc : rec;
                    }
                }
                if (seq >= 1) WAIT(h_free, (seq - 1) & 1);           // every CTA's down products of the previous tile are complete
                if (act && ni_loc < nj) {
                    const int kslot = off + ni_loc;
                    const int p0 = ch * 4 + (isup ? 2 : 0);          // first 16-byte piece (8 tokens) of this lane's 16 tokens
                    unsigned char* rowp = gbase + G::OFF_H + kslot * 128;
#pragma unroll
                    for (int pp = 0; pp < 2; ++pp) {
                        uint32_t hi[4], lo[4];
#pragma unroll
                        for (int e2 = 0; e2 < 4; ++e2) {
                            const float f0 = hv[pp * 8 + 2 * e2], f1 = hv[pp * 8 + 2 * e2 + 1];
                            const __nv_bfloat162 h2 = __floats2bfloat162_rn(f0, f1);
                            const float2 hf = __bfloat1622float2(h2);
                            const __nv_bfloat162 l2 = __floats2bfloat162_rn(f0 - hf.x, f1 - hf.y);
                            hi[e2] = *reinterpret_cast<const uint32_t*>(&h2);
                            lo[e2] = *reinterpret_cast<const uint32_t*>(&l2);
                        }
                        const int o = ((p0 + pp) ^ (kslot & 7)) << 4;
                        *reinterpret_cast<uint4*>(rowp + o) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                        *reinterpret_cast<uint4*>(rowp + H_HALF + o) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                    }
                }
                {
                    // slots from ts to the end of the last product step: zeros (their weight rows are zeros too)
                    const int prow = ts + (et >> 4), pp = et & 15;
                    if (prow < (((ts + 15) >> 4) << 4))
                        *reinterpret_cast<uint4*>(gbase + G::OFF_H + (pp >> 3) * H_HALF + prow * 128 + ((pp & 7) << 4)) = make_uint4(0u, 0u, 0u, 0u);
                }
                fence_proxy_async_smem();
                stop = named_barrier_or(1, 256, gave_up || *sAbort);
                if (et == 0) mbar_arrive_expect_tx(h_full, (uint32_t)(ts - nj) * 256u);
                if (et < 2 * (CS - 1) && nj > 0) {
                    int peer = et >> 1;
                    if (peer >= j) ++peer;
                    const uint32_t src = sH + (et & 1) * H_HALF + off * 128;
                    bulk_copy_to_peer(map_to_rank(src, peer), src, (uint32_t)nj * 128u, map_to_rank(h_full, peer));
                }
                if (et == 0 && i == 0) RM_PS(item, 3);
            }
            if (stop) break;
            if (run.ntiles > 0) {
                // the item's down products are complete: add this CTA's [T x H/8] part to the residual stream
                const int d2b = ND2 == 2 ? (ni & 1) : 0, nu = ND2 == 2 ? (ni >> 1) : ni;
                ++ni;
                WAIT(d2_full(d2b), nu & 1);
                tc_fence_after();
                if (et == 0) RM_PS(item, 5);
                float* rb = a.r + (size_t)b * T * H + j * HS8 + q4 * 32 + lane;
#pragma unroll
                for (int mb = 0; mb < NMB; ++mb) {
                    float hi[32], lo[32];
                    const uint32_t col = tmem + G::D2_COL + d2b * (2 * NTOK) + mb * (2 * NTOK) + ch * 32 + ((uint32_t)(q4 * 32) << 16);
                    tmem_ld32(col, hi);
                    tmem_ld32(col + NTOK, lo);
#pragma unroll
                    for (int r = 0; r < 32; ++r) {
                        const int t = ch * 32 + r;
                        if (t < T) red_add_f32(rb + (size_t)t * H + mb * 128, hi[r] + lo[r]);
                    }
                }
                tc_fence_before();
                mbar_arrive(d2_empty(d2b));
                if (et == 0) RM_PS(item, 6);
                __threadfence();
                stop = named_barrier_or(1, 256, gave_up || *sAbort);
            }
            if (et == 0) { red_release_gpu(a.sync + b, 1); RM_PS(item, 7); }
        }
    }
#undef WAIT
    tc_fence_before();
    __syncthreads();
    cluster_sync();                    // no CTA leaves while a peer may still write into its shared memory
    if (warp == W_MMA) tmem_dealloc(tmem, 512);
}

// ---- host side
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

// bf16 matrix [rows, cols] row-major, boxes of 64 rows x 64 columns, 128-byte swizzle; rows past the extent read as zeros
int make_x_map(CUtensorMap* tm, const void* ptr, uint64_t rows, uint64_t cols) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return RM_ERR_UNSUPPORTED;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * sizeof(__nv_bfloat16)};
    cuuint32_t box[2] = {64, NTOK};
    cuuint32_t es[2] = {1, 1};
    const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? RM_OK : RM_ERR_CUDA;
}

template <int HS8>
int query_clusters(int* out) {
    auto kern = step_kernel<HS8>;
    RM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<HS8>::TOTAL));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CS * 32);
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = Geo<HS8>::TOTAL;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = CS;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    RM_CUDA_TRY(cudaOccupancyMaxActiveClusters(out, kern, &cfg));
    return RM_OK;
}

template <int HS8>
int launch(rm_ctx* ctx, const PArgs& a, const CUtensorMap& tmX, const CUtensorMap& tmXext, int n_clusters, cudaStream_t s) {
    static rm_smem_configured configured = {};
    if (!configured.covers(ctx->device, Geo<HS8>::TOTAL)) {
        RM_CUDA_TRY(cudaFuncSetAttribute(step_kernel<HS8>, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<HS8>::TOTAL));
        configured.set(ctx->device, Geo<HS8>::TOTAL);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_clusters * CS);
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = Geo<HS8>::TOTAL;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = CS;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, step_kernel<HS8>, a, tmX, tmXext));
    ctx->launches++;
    return RM_OK;
}

inline size_t align_up(size_t v, size_t al) { return (v + al - 1) / al * al; }

}  // namespace

int rm_persist_init(rm_ctx* ctx) {
    ctx->persist_clusters = 0;
    ctx->persist_xbuf = nullptr;
    int n = 0, rc = RM_OK;
    if (ctx->g.H == 1024) rc = query_clusters<128>(&n);
    else if (ctx->g.H == 2048) rc = query_clusters<256>(&n);
    else return RM_OK;
    if (rc != RM_OK) return rc;
    ctx->persist_clusters = n;
    return RM_OK;
}

bool rm_persist_supported(const rm_ctx* ctx, int B, int T) {
    const int H = ctx->g.H;
    return (H == 1024 || H == 2048) && T >= 1 && T <= NTOK && B >= 1 && B <= MAXB && ctx->g.L <= MAXL &&
           ctx->persist_clusters > 0 && encode_fn() != nullptr;
}

size_t rm_persist_workspace_bytes(const rm_ctx* ctx) {
    if (ctx->persist_clusters <= 0) return 0;
    return 256 + (size_t)ctx->persist_clusters * 2 * NTOK * ctx->g.H * sizeof(__nv_bfloat16);
}

int rm_persist_debug_stamps(long long* host_out, int n) {
#ifdef RM_PHASE_TIMING
    if (n > 64 * 128 * 16) n = 64 * 128 * 16;
    return cudaMemcpyFromSymbol(host_out, g_ps_stamps, sizeof(long long) * n) == cudaSuccess ? RM_OK : RM_ERR_CUDA;
#else
    (void)host_out; (void)n;
    return RM_ERR_UNSUPPORTED;
#endif
}

int rm_launch_step_persist(rm_ctx* ctx, const rm_step_args& sa, void* ws, cudaStream_t s) {
    const rm_geom& g = ctx->g;
    PArgs a{};
    for (int l = 0; l < sa.L; ++l) a.packed[l] = static_cast<const __nv_bfloat16*>(sa.packed_layers[l]);
    a.r = sa.r;
    a.sync = reinterpret_cast<int*>(ws);
    a.xbuf = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(ws) + 256);
    a.idx = sa.idx;
    a.count = sa.count;
    a.idx_b_stride = sa.idx_b_stride;
    a.idx_l_stride = sa.idx_l_stride;
    a.list_cap = sa.list_cap;
    a.count_b_stride = sa.count_b_stride;
    a.record = sa.record;
    a.rec_b_stride = sa.rec_b_stride;
    a.record_scale = sa.record_scale;
    a.status = ctx->d_status;
    a.L = sa.L;
    a.B = sa.B;
    a.T = sa.T;
    a.I = g.I;
    a.x_ext = sa.x_ext ? 1 : 0;
    int nc = ctx->persist_clusters;
    if (ctx->max_clusters_override > 0 && ctx->max_clusters_override < nc) nc = ctx->max_clusters_override;
    if (ctx->persist_xbuf != a.xbuf) {
        const int rc = make_x_map(reinterpret_cast<CUtensorMap*>(ctx->persist_tm), a.xbuf,
                                  (uint64_t)ctx->persist_clusters * 2 * NTOK, (uint64_t)g.H);
        if (rc != RM_OK) return rc;
        ctx->persist_xbuf = a.xbuf;
    }
    alignas(64) CUtensorMap tm_ext;
    if (sa.x_ext) {
        const int rc = make_x_map(&tm_ext, sa.x_ext, (uint64_t)sa.T, (uint64_t)g.H);
        if (rc != RM_OK) return rc;
    } else {
        tm_ext = *reinterpret_cast<const CUtensorMap*>(ctx->persist_tm);
    }
    RM_CUDA_TRY(cudaMemsetAsync(a.sync, 0, 256, s));
    const CUtensorMap& tmX = *reinterpret_cast<const CUtensorMap*>(ctx->persist_tm);
    return g.H == 1024 ? launch<128>(ctx, a, tmX, tm_ext, nc, s) : launch<256>(ctx, a, tmX, tm_ext, nc, s);
}
