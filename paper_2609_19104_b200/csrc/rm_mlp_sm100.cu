// Fused masked gated-MLP layer for sm_100a: one kernel per layer, thread-block clusters of 8 CTAs.
//
// Decomposition.  The active neurons of a layer are cut into tiles of 64; a cluster owns a contiguous run of
// tiles.  CTA j of the cluster owns column slice j (Hs = H/8 columns) of the model dimension for BOTH projections:
//   gate/up : D1[128 x T] = [64 gate rows ; 64 up rows](slice j) . x(slice j)^T      partial over the H split
//   exchange: partial sums are reduce-scattered through distributed shared memory (CTA o receives the rows of
//             tile neurons 8o..8o+7), the owner applies GeLU-tanh(g) * u and broadcasts h to the 8 CTAs as a
//             bf16 hi + lo pair (h = hi + lo to 2^-17, so the tensor-core product keeps fp32-level accuracy)
//   down    : D2[Hs x T] += Wd(slice j, tile) as an MN-major operand . (h_hi + h_lo)^T   accumulated in TMEM
// so a neuron's 3*Hs*2 contiguous bytes are read exactly once by exactly one CTA, x is never replicated inside a
// cluster, and h never leaves the chip.  Both products run on the 5th-generation tensor cores (tcgen05.mma,
// accumulators in tensor memory); gathered rows are placed by 16-byte cp.async directly into the 128-byte
// swizzled operand layout, one cp.async group per tile half, so the next tile's weights stream in while the
// current tile is in its exchange phases.  At the end of an episode each CTA adds its [T x Hs] partial of y to
// the fp32 residual stream with red.global.add.
//
// Layers are chained with programmatic dependent launch: a layer's CTAs become resident, set up, issue the loads
// of their first tile (weight addresses depend only on the index lists) and then wait (griddepcontrol.wait) for
// the previous layer's atomics before touching activations.
#include <cuda.h>
#include <cstdio>
#include <cstdlib>

#include "rm_common.cuh"
#include "rm_sm100.cuh"

using namespace sm100;

// Optional phase timing (build with -DRM_PHASE_TIMING): thread 0 of every CTA stamps clock64() at phase
// boundaries of its first tile into a device buffer that rm_debug_phase_times copies out.
#ifdef RM_PHASE_TIMING
__device__ long long g_phase_stamps[256 * 32];
#define RM_STAMP(k)                                                                                              \
    do {                                                                                                         \
        if (threadIdx.x == 0 && blockIdx.x < 256 && stamp_ok) g_phase_stamps[blockIdx.x * 32 + (k)] = clock64(); \
    } while (0)
__device__ __forceinline__ long long rm_globaltimer() {
    long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// wall-clock (ns) stamps per launch: slot = launch sequence number taken from a device counter
__device__ long long g_wall_stamps[64 * 256 * 4];
__device__ int g_wall_seq;
#define RM_WALL(k)                                                                                          \
    do {                                                                                                    \
        if (threadIdx.x == 0 && blockIdx.x < 256) g_wall_stamps[((wall_seq & 63) * 256 + blockIdx.x) * 4 + (k)] = rm_globaltimer(); \
    } while (0)
// warp-specialised kernel: globaltimer per (CTA < 16, tile < 16, event < 8), written by each role's first thread
__device__ long long g_ws_stamps[16 * 16 * 16];
#define RM_WS(tile, ev)                                                                                   \
    do {                                                                                                  \
        if (blockIdx.x < 16 && (tile) < 16) g_ws_stamps[(blockIdx.x * 16 + (tile)) * 16 + (ev)] = rm_globaltimer(); \
    } while (0)
#else
#define RM_STAMP(k) do { } while (0)
#define RM_WALL(k) do { } while (0)
#define RM_WS(tile, ev) do { } while (0)
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
    int p_row;                     // floats per row of the partial-sum exchange buffer
    int add_residual;              // r_in is added into r_out (spread over all CTAs)
    int* status;
    int wall_seq;                  // launch sequence number (phase-timing builds only)
    int l2_prefetch;               // tiles of L2 prefetch distance in the warp-specialised kernel (0: off)
    // anchor-relative update (Eq. 4): see rm_layer_args
    int anchor_mode;
    float* y_anchor;
    float* h_anchor;
    int64_t h_stride;
    const float* gate;
};

// r_out[0..3] += r[0..3] (+ gate * y_anchor in an update step, Eq. 4): the residual part of a layer's output.
// ya_update is the layer's y_anchor in update steps, else NULL.
__device__ __forceinline__ void add_residual4(const float* ya_update, const float* gate, int H, float* o,
                                              size_t off_bt_h, int col, int b, float r0, float r1, float r2, float r3) {
    if (ya_update) {
        const float4 ya = *reinterpret_cast<const float4*>(ya_update + off_bt_h + col);
        float4 g = make_float4(1.f, 1.f, 1.f, 1.f);
        if (gate) g = *reinterpret_cast<const float4*>(gate + (size_t)b * H + col);
        r0 = fmaf(g.x, ya.x, r0); r1 = fmaf(g.y, ya.y, r1); r2 = fmaf(g.z, ya.z, r2); r3 = fmaf(g.w, ya.w, r3);
    }
    red_add_v4(o, r0, r1, r2, r3);
}

// floats per row of the exchange buffer: T rounded up to 4 with an odd number of 16-byte chunks, so that the
// eight rows written by one warp-store fall into distinct bank groups
__host__ __device__ constexpr int p_row_for(int T) { return 4 * (((T + 3) / 4) | 1); }

// A wait that ran out of polls records the source line of the wait and the CTA (readable as "status_detail").
#define wait_bar(bar, parity) wait_bar_at((bar), (parity), __LINE__)

// Adds one warp's share of a CTA's [T x Hs] down-projection partial (fp32 in tensor memory, lanes = output columns)
// to the episode's residual stream, times the output gate; the anchor step of Eq. 4 also accumulates the ungated
// partial into y_anchor.  Pointers are already offset to the episode.  wrow: which 32-lane quarter of the accumulator
// this warp reads; token columns c0_first, c0_first + c0_step, ...
// Width in tensor-memory columns of one 128-row block of the down accumulator.  At H = 2048 with 64-token tiles the
// product is issued once per K step against the operand [h_hi | h_lo] (N = 128: the two h tiles lie one
// leading-dimension step apart), so the block holds Wd*h_hi in columns 0..63 and Wd*h_lo in columns 64..127 and
// readers add the halves; that halves the number of down-product instructions, which bound the tile rate there.
// Elsewhere (H = 1024, where the lean kernel must stay within 128 registers and the products are not the limit, and
// 32-token tiles) two N = NTOK products accumulate into one block.
__host__ __device__ constexpr bool d2_wide(int ntok, int hs) { return ntok == 64 && hs == 256; }
__host__ __device__ constexpr int d2_width(int ntok, int hs) { return d2_wide(ntok, hs) ? 128 : ntok; }
template <int NTOK, int HS>
__device__ __forceinline__ void ld_d2(uint32_t taddr, float (&v)[32]) {
    tmem_ld32(taddr, v);
    if (d2_wide(NTOK, HS)) {
        float w[32];
        tmem_ld32(taddr + NTOK, w);
#pragma unroll
        for (int k = 0; k < 32; ++k) v[k] += w[k];
    }
}

template <int NTOK, int HS>
__device__ __noinline__ void flush_partial(float* __restrict__ r_out, float* __restrict__ y_anchor,
                                           const float* __restrict__ gate, bool write_anchor, uint32_t tmem_d2, int wrow,
                                           int lane, int c0_first, int c0_step, int T, int H, int col_base) {
#pragma unroll
    for (int mm = 0; mm < HS / 128; ++mm) {
        const int col = col_base + mm * 128 + wrow * 32 + lane;
        const float gc = gate ? gate[col] : 1.f;
        for (int c0 = c0_first; c0 < NTOK; c0 += c0_step) {
            float v[32];
            ld_d2<NTOK, HS>(tmem_d2 + mm * d2_width(NTOK, HS) + ((uint32_t)(wrow * 32) << 16) + c0, v);
            // explicit red.global.add: with the gate factor in front, atomicAdd() compiled to something far slower
            // here (measured: 60 against 37 us per H = 2048 layer)
            if (write_anchor) {
#pragma unroll
                for (int k = 0; k < 32; ++k)
                    if (c0 + k < T) red_add_f32(y_anchor + (size_t)(c0 + k) * H + col, v[k]);
            }
#pragma unroll
            for (int k = 0; k < 32; ++k)
                if (c0 + k < T) red_add_f32(r_out + (size_t)(c0 + k) * H + col, gc * v[k]);
        }
    }
}

// The same accumulator, scaled by the gate, laid out in shared memory as [128-column block][token][128 columns] for
// the copy engine's bulk add (one box of the [B, T, H] tensor map per block).  Out of line for the same reason.
template <int NTOK, int HS>
__device__ __noinline__ void stage_partial(float* __restrict__ stage, const float* __restrict__ gate, uint32_t tmem_d2,
                                           int wrow, int lane, int c0_first, int c0_step, int T, int col_base) {
#pragma unroll
    for (int mm = 0; mm < HS / 128; ++mm) {
        const int cl = wrow * 32 + lane;
        const float gc = gate ? gate[col_base + mm * 128 + cl] : 1.f;
        for (int c0 = c0_first; c0 < NTOK; c0 += c0_step) {
            float v[32];
            ld_d2<NTOK, HS>(tmem_d2 + mm * d2_width(NTOK, HS) + ((uint32_t)(wrow * 32) << 16) + c0, v);
#pragma unroll
            for (int k = 0; k < 32; ++k)
                if (c0 + k < T) stage[(mm * NTOK + c0 + k) * 128 + cl] = gc * v[k];
        }
    }
}

template <int NTOK, int HS, bool PIPE>
struct Smem {
    static constexpr int KB = HS / 64;                       // 64-column (128-byte) blocks per slice
    static constexpr int NB = PIPE ? 2 : 1;                  // buffers of the exchange state (tiles in flight)
    static constexpr bool STAGED = PIPE && HS == 128;        // dedicated staging area for the outgoing partial sums
    static constexpr int X_BYTES = KB * NTOK * 128;
    static constexpr int GU_STAGE = KB * 128 * 128;
    static constexpr int DN_STAGE = KB * NT * 128;
    static constexpr int HT_HALF = NT * 128;                 // 8 atoms of [8 neurons x 64 tokens] bf16
    static constexpr int OFF_X = 0;
    static constexpr int OFF_GU = OFF_X + X_BYTES;
    static constexpr int OFF_DN = OFF_GU + GU_STAGE;
    static constexpr int OFF_HT = OFF_DN + DN_STAGE;         // per buffer: hi tile, then lo tile
    static constexpr int OFF_HS = OFF_HT + NB * 2 * HT_HALF; // per buffer: this CTA's h atom (1 KB hi, 1 KB lo)
    static constexpr int OFF_SS = OFF_HS + NB * 2048;        // [CS][64] floats: row sums of squares per source CTA
    static constexpr int OFF_N = OFF_SS + CS * 64 * 4;       // [2][64] neuron ids of two consecutive tiles
    static constexpr int OFF_PREF = OFF_N + 2 * NT * 4;      // [MAXB+1] tile prefix, [MAXB] counts
    static constexpr int OFF_BAR = ((OFF_PREF + (2 * MAXB + 1) * 4 + 7) / 8) * 8;
    static constexpr int OFF_P = ((OFF_BAR + 96 + 15) / 16) * 16;   // NB x [CS][16][p_row] floats (+ staging), sized at launch
    static constexpr int TMEM_COLS_USED = NB * NTOK + (HS / 128) * d2_width(NTOK, HS);
    static constexpr int TMEM_COLS = TMEM_COLS_USED <= 32 ? 32 : TMEM_COLS_USED <= 64 ? 64 :
                                     TMEM_COLS_USED <= 128 ? 128 : TMEM_COLS_USED <= 256 ? 256 : 512;
    static int total_bytes(int T) { return OFF_P + (NB + (STAGED ? 1 : 0)) * CS * 16 * p_row_for(T) * 4 + 1024; }
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

struct TileRef {
    int b, p0, nvalid;
    bool first, last;              // first / last tile of its episode within this cluster's run
};

// EQ4 = false compiles the anchor-relative update and the output gate out (the zero-fill step pays nothing for them)
template <int NTOK, int HS, bool PIPE, bool EQ4>
__global__ void __launch_bounds__(FT, (HS == 128 && !PIPE ? 2 : 1)) fused_layer_kernel(const FusedArgs a,
                                                                                               const __grid_constant__ CUtensorMap tmOut) {
    const int anchor_mode = EQ4 ? a.anchor_mode : (int)RM_ANCHOR_NONE;
    const float* const gate = EQ4 ? a.gate : nullptr;
    const float* const ya_update = anchor_mode == RM_ANCHOR_UPDATE ? a.y_anchor : nullptr;
    using S = Smem<NTOK, HS, PIPE>;
    constexpr int NB = S::NB;
    constexpr int KB = S::KB;
    extern __shared__ unsigned char smem_dyn[];
    // 1024-byte alignment: the 128-byte swizzle is a function of absolute shared-memory address bits
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* gbase = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t sX = base + S::OFF_X, sGU = base + S::OFF_GU, sDN = base + S::OFF_DN, sHT = base + S::OFF_HT;
    const uint32_t sP = base + S::OFF_P, sSS = base + S::OFF_SS;
    const float* gSS = reinterpret_cast<const float*>(gbase + S::OFF_SS);
    int* gN = reinterpret_cast<int*>(gbase + S::OFF_N);
    int* gPref = reinterpret_cast<int*>(gbase + S::OFF_PREF);
    int* gCnt = gPref + MAXB + 1;
    // mbarriers: MMA completion (gate/up per buffer, down) and arrival of the exchanges (partial sums and h per
    // buffer, sums of squares)
    const uint32_t bar0 = base + S::OFF_BAR;
    const uint32_t bar_dn = bar0 + 48, bar_s = bar0 + 56, s_tmem = bar0 + 64;
    auto bar_gu = [&](int pb) { return bar0 + 8 * pb; };
    auto bar_p = [&](int pb) { return bar0 + 16 + 8 * pb; };
    auto bar_h = [&](int pb) { return bar0 + 32 + 8 * pb; };
    volatile uint32_t* g_tmem = reinterpret_cast<volatile uint32_t*>(gbase + S::OFF_BAR + 64);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef RM_PHASE_TIMING
    bool stamp_ok = true;
#endif
    RM_STAMP(0);
#ifdef RM_PHASE_TIMING
    const int wall_seq = a.wall_seq;
#endif
    RM_WALL(0);
    const int j = (int)cluster_ctarank();
    const int cid = (int)cluster_id_x(), NC = (int)cluster_count_x();
    const int H = a.H, T = a.T, PR = a.p_row;

    // ---- set-up: barriers, tensor memory, per-episode tile counts
    if (tid == 0) {
        for (int pb = 0; pb < 2; ++pb) { mbar_init(bar_gu(pb), 1); mbar_init(bar_p(pb), 1); mbar_init(bar_h(pb), 1); }
        mbar_init(bar_dn, 1);
        mbar_init(bar_s, 1);
        fence_mbar_init();
        int acc = 0;
        const int cap = (int)(a.list_cap < (int64_t)a.I ? a.list_cap : (int64_t)a.I);
        for (int b = 0; b < a.B; ++b) {
            int c = a.I;                   // dense: every neuron
            if (a.count) {                 // a list, or (no list) the leading `count` neurons of a compact layer
                c = a.count[(size_t)b * a.count_stride];
                if (c < 0 || c > cap) { rm_set_status(a.status, RM_ERR_INDEX); c = c < 0 ? 0 : cap; }
            }
            gCnt[b] = c;
            gPref[b] = acc;
            acc += (c + NT - 1) / NT;
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
    const uint32_t tmem_d2 = tmem_d1 + NB * NTOK;
    RM_STAMP(1);

    // this cluster's run of tiles
    const int tiles_total = gPref[a.B];
    const int n_active = tiles_total < NC ? tiles_total : NC;
    const int g_lo = cid < n_active ? (int)((long long)cid * tiles_total / n_active) : 0;
    const int g_hi = cid < n_active ? (int)((long long)(cid + 1) * tiles_total / n_active) : 0;
    // The next layer may become resident once every CTA of this one has said so.  Its CTAs then set up and gather their
    // first tile on the same SMs, which slows whatever runs there (measured: +1.1 us on the x preparation of the
    // clusters it hits), and with few clusters per layer a third layer piles in behind it.  So in launches of up to 16
    // clusters a CTA with work says so only once its slice of the residual has arrived (inside the x preparation); the
    // next layer still has the rest of this one to get ready.  With more clusters the next layer finds no free SM
    // before this one ends anyway, and the early release measured 2-3 % better.
    bool pdl_fired = false;
    if (g_lo >= g_hi || a.x || n_active > 16) { pdl_launch_dependents(); pdl_fired = true; }

    auto tile_ref = [&](int g) {
        TileRef r;
        int b = 0;
        while (gPref[b + 1] <= g) ++b;
        r.b = b;
        r.p0 = (g - gPref[b]) * NT;
        const int left = gCnt[b] - r.p0;
        r.nvalid = left < NT ? left : NT;
        r.first = (g == g_lo) || (g == gPref[b]);
        r.last = (g == g_hi - 1) || (g == gPref[b + 1] - 1);
        return r;
    };

    // per-thread share of a tile's gather: rows q0 = tid/8 and q0 + 32 of the tile, 16-byte chunk ch = tid%8
    const int q0 = tid >> 3, ch = tid & 7;
    const __nv_bfloat16* slice = a.packed + (size_t)j * 3 * HS + ch * 8;
    auto neuron_of = [&](const TileRef& r, int q) {
        int n = -1;
        if (q < r.nvalid) {
            n = a.idx ? a.idx[(size_t)r.b * a.idx_stride + r.p0 + q] : r.p0 + q;
            if (n < 0 || n >= a.I) { rm_set_status(a.status, RM_ERR_INDEX); n = -1; }
        }
        return n;
    };
    // gate and up rows of tile g into GU stage `st`: rows q (gate) and 64+q (up), swizzled 128-byte rows
    auto issue_gu = [&](int g) {
        const TileRef r = tile_ref(g);
        const int n0 = neuron_of(r, q0), n1 = neuron_of(r, q0 + 32);
        if (ch == 0) { gN[((g - g_lo) & 1) * NT + q0] = n0; gN[((g - g_lo) & 1) * NT + q0 + 32] = n1; }
        const __nv_bfloat16* s0 = slice + (size_t)(n0 < 0 ? 0 : n0) * 3 * H;
        const __nv_bfloat16* s1 = slice + (size_t)(n1 < 0 ? 0 : n1) * 3 * H;
        const uint32_t d0 = sGU + q0 * 128 + ((ch ^ (q0 & 7)) << 4);   // (q0+32)&7 == q0&7
#pragma unroll
        for (int kb = 0; kb < KB; ++kb) {
            cp_async16(d0 + kb * 16384, s0 + kb * 64, n0 >= 0);                           // gate, neuron q0
            cp_async16(d0 + kb * 16384 + 32 * 128, s1 + kb * 64, n1 >= 0);                // gate, neuron q0+32
            cp_async16(d0 + kb * 16384 + 64 * 128, s0 + HS + kb * 64, n0 >= 0);           // up, neuron q0
            cp_async16(d0 + kb * 16384 + 96 * 128, s1 + HS + kb * 64, n1 >= 0);           // up, neuron q0+32
        }
    };
    // down rows of tile g into DN stage `st`: MN-major operand, 64 neurons x 128 bytes per 64-column block
    auto issue_dn = [&](int g) {
        const TileRef r = tile_ref(g);
        const int n0 = neuron_of(r, q0), n1 = neuron_of(r, q0 + 32);
        const __nv_bfloat16* s0 = slice + (size_t)(n0 < 0 ? 0 : n0) * 3 * H + 2 * HS;
        const __nv_bfloat16* s1 = slice + (size_t)(n1 < 0 ? 0 : n1) * 3 * H + 2 * HS;
        const uint32_t d0 = sDN + q0 * 128 + ((ch ^ (q0 & 7)) << 4);
#pragma unroll
        for (int cb = 0; cb < KB; ++cb) {
            cp_async16(d0 + cb * 8192, s0 + cb * 64, n0 >= 0);
            cp_async16(d0 + cb * 8192 + 32 * 128, s1 + cb * 64, n1 >= 0);
        }
    };

    __syncthreads();                       // gPref / gCnt
    // ---- prologue: the first tile's weights start streaming before the previous layer has finished
    if (g_lo < g_hi) issue_gu(g_lo);
    cp_async_commit();
    if (g_lo < g_hi) issue_dn(g_lo);
    cp_async_commit();

    // Which of the clusters that work on an episode adds which token rows of the residual (see xprep).  Integer
    // divisions: ~0.8 us, so the first episode's answer is worked out here, before the dependency wait.
    auto residual_share = [&](int b, int& n_share, int& my_share) {
        const long long e0 = gPref[b], e1 = gPref[b + 1];                  // tile range of the episode
        // cluster c owns tiles [c*tt/na, (c+1)*tt/na); first cluster with hi > e0, last with lo < e1
        int first_c = (int)((e0 * n_active) / tiles_total);
        while ((long long)(first_c + 1) * tiles_total / n_active <= e0) ++first_c;
        int last_c = (int)(((e1 - 1) * n_active) / tiles_total);
        while (last_c + 1 < n_active && (long long)(last_c + 1) * tiles_total / n_active < e1) ++last_c;
        n_share = last_c - first_c + 1;
        my_share = cid - first_c;
    };
    int share_b = -1, share_n = 1, share_my = 0;
    if (a.add_residual && g_lo < g_hi) {
        share_b = tile_ref(g_lo).b;
        residual_share(share_b, share_n, share_my);
    }

    RM_WALL(1);
    pdl_wait();                            // the previous layer's output is complete and visible
    RM_STAMP(2);
    RM_WALL(2);

    RM_STAMP(3);

    uint32_t par_dn = 0, par_s = 0;
    constexpr uint32_t IDESC_GU = idesc_bf16_f32(128, NTOK, false, false);
    constexpr uint32_t IDESC_DN = idesc_bf16_f32(128, d2_width(NTOK, HS), true, true);
    const uint64_t desc_k = smem_desc_sw128(0, 16, 1024);        // K-major operand: 8-row groups 1024 B apart
    const uint64_t desc_mn = smem_desc_sw128(0, 8192, 1024);     // MN-major operand: 64-element blocks 8192 B apart
    const int n_tiles = g_hi - g_lo;
    const int p_bytes = CS * 16 * PR * 4;                        // one exchange buffer
    int cur_b = -1;
    // buffer and barrier phase of local tile i (every second tile reuses a buffer when two are in flight)
    auto buf_of = [&](int i) { return PIPE ? (i & 1) : 0; };
    auto phase_of = [&](int i) { return (uint32_t)(PIPE ? ((i >> 1) & 1) : (i & 1)); };
    bool gave_up = false;
    auto wait_bar_at = [&](uint32_t bar, uint32_t parity, int line) {
        if (!mbar_wait(bar, parity)) {
            rm_set_status_at(a.status, RM_ERR_TIMEOUT, (line << 12) | (int)(blockIdx.x & 0xfffu));
            gave_up = true;
        }
    };

    // ---- phase: x slice of episode b -> bf16, 128-byte-swizzled K-major operand tile (cluster-collective)
    auto xprep = [&](int b) {
        cur_b = b;
        constexpr int PARTS = FT / NTOK;                   // threads per token row
        constexpr int CPP = HS / PARTS;                    // columns per thread
        const int t = tid / PARTS, part = tid % PARTS;
        // clusters whose runs contain tiles of this episode share the addition of its residual rows
        int n_share = 1, my_share = 0;
        if (a.add_residual) {
            if (b == share_b) { n_share = share_n; my_share = share_my; }
            else residual_share(b, n_share, my_share);
        }
        if (a.x) {
            const uint4* src = reinterpret_cast<const uint4*>(a.x + ((size_t)b * T + t) * H + (size_t)j * HS + part * CPP);
#pragma unroll
            for (int i = 0; i < CPP / 8; ++i) {
                const uint4 u = t < T ? src[i] : make_uint4(0, 0, 0, 0);
                const int k = part * CPP + i * 8;
                *reinterpret_cast<uint4*>(gbase + S::OFF_X + (k >> 6) * (NTOK * 128) + t * 128 +
                                          ((((k & 63) >> 3) ^ (t & 7)) << 4)) = u;
            }
        } else {
            float v[CPP];
            float ss = 0.f;
            if (t < T) {
                const float4* src = reinterpret_cast<const float4*>(a.r_in + ((size_t)b * T + t) * H + (size_t)j * HS + part * CPP);
#pragma unroll
                for (int i = 0; i < CPP / 4; ++i) {
                    const float4 f = src[i];
                    v[4 * i] = f.x; v[4 * i + 1] = f.y; v[4 * i + 2] = f.z; v[4 * i + 3] = f.w;
                }
#pragma unroll
                for (int i = 0; i < CPP; ++i) ss = fmaf(v[i], v[i], ss);
            } else {
#pragma unroll
                for (int i = 0; i < CPP; ++i) v[i] = 0.f;
            }
#pragma unroll
            for (int d = 1; d < PARTS; d <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
            if (!pdl_fired) { pdl_launch_dependents(); pdl_fired = true; }   // the residual slice has arrived
            // all-gather of the row sums of squares: the PARTS lanes of a row share the 8 destinations
            if (tid == 0) mbar_arrive_expect_tx(bar_s, CS * NTOK * 4);
#pragma unroll
            for (int dst = part; dst < CS; dst += PARTS)
                st_async_f32(map_to_rank(sSS + (j * 64 + t) * 4, dst), ss, map_to_rank(bar_s, dst));
            // residual: token row t of this episode is added by exactly one of the clusters that work on the
            // episode, from the values already in registers, while the exchange is in flight
            if (a.add_residual && t < T && (t % n_share) == my_share) {
                const size_t row = ((size_t)b * T + t) * H;
                const int col = j * HS + part * CPP;
#pragma unroll
                for (int i = 0; i < CPP / 4; ++i)
                    add_residual4(ya_update, gate, H, a.r_out + row + col + 4 * i, row, col + 4 * i, b, v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            }
            wait_bar(bar_s, par_s);
            par_s ^= 1;
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
        RM_STAMP(4);
    };

    // ---- phase: open local tile i (announce the bytes its two exchanges deliver here; new episode -> new x)
    // Bytes of partial sums a tile delivers to each owner.  The bulk-copy route moves whole padded rows; the
    // per-thread stores send only the columns that exist in tensor memory (the row pad can exceed the token tile).
    const int p_cols = PR < NTOK ? PR : NTOK;
    auto p_tx_bytes = [&](int i) {
        const bool bulk = S::STAGED || (!(i + 1 < n_tiles) && p_bytes <= S::GU_STAGE);
        return bulk ? p_bytes : CS * 16 * p_cols * 4;
    };
    auto open_tile = [&](int i) {
        if (tid == 0) {
            mbar_arrive_expect_tx(bar_p(buf_of(i)), p_tx_bytes(i));
            mbar_arrive_expect_tx(bar_h(buf_of(i)), CS * 2048);
        }
        const TileRef tr = tile_ref(g_lo + i);
        if (tr.b != cur_b) xprep(tr.b);
    };

    // ---- phase: gate/up partial products of tile i over this CTA's column slice (operands are in shared memory
    // and a CTA-wide barrier has made them visible)
    auto mma_gu = [&](int i) {
        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    mma_bf16_ss(tmem_d1 + buf_of(i) * NTOK, desc_k | desc_addr(sGU + kb * 16384 + ks * 32),
                                desc_k | desc_addr(sX + kb * (NTOK * 128) + ks * 32), IDESC_GU, (kb | ks) != 0);
            mma_commit(bar_gu(buf_of(i)));
        }
    };

    // ---- phase: reduce-scatter of tile i.  Row m of D1 (gate or up of tile neuron q) goes to the CTA that owns q.
    // When a staging area is free (the dedicated one, or the gate/up stage when no further tile will refill it) the
    // rows are laid out per destination in local shared memory and moved by 8 bulk copies; otherwise every thread
    // sends its row with asynchronous 16-byte stores.  `refill` says whether the gate/up stage is being refilled.
    auto scatter = [&](int i, bool refill) {
        const int pb = buf_of(i);
        const uint32_t d1 = tmem_d1 + pb * NTOK;
        const bool stage_in_gu = !refill && p_bytes <= S::GU_STAGE;
        if (S::STAGED || stage_in_gu) {
            unsigned char* stg = S::STAGED ? gbase + S::OFF_P + NB * p_bytes : gbase + S::OFF_GU;
            for (int c0 = (warp >> 2) * 32; c0 < NTOK; c0 += 64) {
                float v[32];
                const int m = (warp & 3) * 32 + lane;
                tmem_ld32(d1 + ((uint32_t)((warp & 3) * 32) << 16) + c0, v);
                const int q = m & 63;
                float* row = reinterpret_cast<float*>(stg) + (((q >> 3) * 16 + (m >> 6) * 8 + (q & 7)) * PR + c0);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (c0 + 4 * k < PR)
                        *reinterpret_cast<float4*>(row + 4 * k) = make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
            }
            tc_fence_before();
            fence_proxy_async_smem();
            __syncthreads();
            if (tid < CS)
                bulk_copy_to_peer(map_to_rank(sP + pb * p_bytes + (j * 16 * PR) * 4, tid), smem_u32(stg) + tid * 16 * PR * 4,
                                  16 * PR * 4, map_to_rank(bar_p(pb), tid));
        } else {
            for (int c0 = (warp >> 2) * 32; c0 < NTOK; c0 += 64) {
                float v[32];
                const int m = (warp & 3) * 32 + lane;
                tmem_ld32(d1 + ((uint32_t)((warp & 3) * 32) << 16) + c0, v);
                const int q = m & 63;
                const uint32_t dst = map_to_rank(sP + pb * p_bytes + ((j * 16 + (m >> 6) * 8 + (q & 7)) * PR + c0) * 4, q >> 3);
                const uint32_t rbar = map_to_rank(bar_p(pb), q >> 3);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (c0 + 4 * k < PR) st_async_v4(dst + k * 16, v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3], rbar);
            }
            tc_fence_before();
        }
        RM_STAMP(8);
    };

    // ---- phase: owner work of tile i -- sum the 8 partials, GeLU-tanh(g) * u, activation record, h = hi + lo in
    // bf16 as this CTA's atom of the MN-major h operand, then all-gather the atom into every CTA (bulk copies)
    constexpr int TPL = NTOK / 32;                         // owner work: tokens per lane
    // Eq. 4 update steps: the anchor's h for this lane's tokens of its neuron of tile i.  Requested as soon as the
    // tile's neuron ids are in shared memory, long before the partial sums arrive.
    auto anchor_prefetch = [&](int i, const TileRef& tr, float (&ha_pre)[TPL]) {
#pragma unroll
        for (int k = 0; k < TPL; ++k) ha_pre[k] = 0.f;
        if (anchor_mode != RM_ANCHOR_UPDATE) return;
        const int n = gN[(i & 1) * NT + j * 8 + warp];
        const int t0 = lane * TPL;
        if (n >= 0 && t0 < T) {
            const float* hap = a.h_anchor + ((size_t)tr.b * a.I + n) * a.h_stride + t0;
            if (TPL == 2) { const float2 f = *reinterpret_cast<const float2*>(hap); ha_pre[0] = f.x; ha_pre[TPL - 1] = f.y; }
            else ha_pre[0] = *hap;
#pragma unroll
            for (int k = 0; k < TPL; ++k) if (t0 + k >= T) ha_pre[k] = 0.f;
        }
    };
    auto reduce_bcast = [&](int i, const TileRef& tr, const float (&ha_pre)[TPL]) {
        const int pb = buf_of(i);
        const int ql = warp;                               // local neuron 0..7 (tile neuron 8j + ql)
        const int t0 = lane * TPL;
        const float* gP = reinterpret_cast<const float*>(gbase + S::OFF_P + pb * p_bytes);
        unsigned char* gHS = gbase + S::OFF_HS + pb * 2048;
        float gsum[TPL], usum[TPL];
#pragma unroll
        for (int k = 0; k < TPL; ++k) gsum[k] = usum[k] = 0.f;
        if (t0 < PR) {
#pragma unroll
            for (int src = 0; src < CS; ++src) {
                const float* pg = gP + (src * 16 + ql) * PR + t0;
                const float* pu = gP + (src * 16 + 8 + ql) * PR + t0;
#pragma unroll
                for (int k = 0; k < TPL; ++k) { gsum[k] += pg[k]; usum[k] += pu[k]; }
            }
        }
        float rec = 0.f;
        float hv[TPL];
#pragma unroll
        for (int k = 0; k < TPL; ++k) {
            hv[k] = (t0 + k < T) ? rm_gelu_tanh(gsum[k]) * usum[k] : 0.f;
            rec += fabsf(hv[k]);
        }
        // Eq. 4: the anchor step retains h; a later step sends its difference from the anchor's h down the projection
        if (anchor_mode != RM_ANCHOR_NONE) {
            const int n = gN[(i & 1) * NT + j * 8 + ql];
            if (n >= 0 && t0 < T) {
                float* hap = a.h_anchor + ((size_t)tr.b * a.I + n) * a.h_stride + t0;
                if (anchor_mode == RM_ANCHOR_WRITE) {
                    if (TPL == 2) *reinterpret_cast<float2*>(hap) = make_float2(hv[0], hv[TPL - 1]);
                    else *hap = hv[0];
                } else {
#pragma unroll
                    for (int k = 0; k < TPL; ++k) hv[k] -= ha_pre[k];
                }
            }
        }
        // row = local neuron, 128 bytes = 64 tokens, 16-byte chunks swizzled by the row; hi at 0, lo at 1024
        {
            unsigned char* rowp = gHS + ql * 128 + ((((t0 >> 3) ^ ql) & 7) << 4) + (t0 & 7) * 2;
            if (TPL == 2) {
                const __nv_bfloat162 hi = __floats2bfloat162_rn(hv[0], hv[TPL - 1]);
                const float2 hf = __bfloat1622float2(hi);
                const __nv_bfloat162 lo = __floats2bfloat162_rn(hv[0] - hf.x, hv[TPL - 1] - hf.y);
                *reinterpret_cast<__nv_bfloat162*>(rowp) = hi;
                *reinterpret_cast<__nv_bfloat162*>(rowp + 1024) = lo;
            } else {
                const __nv_bfloat16 hi = __float2bfloat16_rn(hv[0]);
                *reinterpret_cast<__nv_bfloat16*>(rowp) = hi;
                *reinterpret_cast<__nv_bfloat16*>(rowp + 1024) = __float2bfloat16_rn(hv[0] - __bfloat162float(hi));
            }
        }
        if (a.record) {
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) rec += __shfl_xor_sync(0xffffffffu, rec, d);
            const int n = gN[(i & 1) * NT + j * 8 + ql];
            if (lane == 0 && n >= 0)
                a.record[(size_t)tr.b * a.record_stride + n] = a.record_scale ? rec * a.record_scale[n] : rec;
        }
        fence_proxy_async_smem();
        __syncthreads();
        if (tid < 2 * CS) {
            const int dst = tid >> 1, part = tid & 1;
            bulk_copy_to_peer(map_to_rank(sHT + pb * 2 * S::HT_HALF + part * S::HT_HALF + j * 1024, dst),
                              smem_u32(gHS) + part * 1024, 1024, map_to_rank(bar_h(pb), dst));
        }
        RM_STAMP(10);
    };

    // ---- phase: down projection of tile i, accumulated in tensor memory across the episode's tiles
    auto mma_dn = [&](int i, const TileRef& tr) {
        if (tid == 0) {
            fence_proxy_async_smem();
            tc_fence_after();
            const uint32_t ht = sHT + buf_of(i) * 2 * S::HT_HALF;
#pragma unroll
            for (int mm = 0; mm < HS / 128; ++mm)
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint64_t aa = desc_mn | desc_addr(sDN + mm * 16384 + ks * 2048);
                    mma_bf16_ss(tmem_d2 + mm * d2_width(NTOK, HS), aa, desc_mn | desc_addr(ht + ks * 2048), IDESC_DN,
                                !(tr.first && ks == 0));
                    if (!d2_wide(NTOK, HS))
                        mma_bf16_ss(tmem_d2 + mm * NTOK, aa, desc_mn | desc_addr(ht + S::HT_HALF + ks * 2048), IDESC_DN, true);
                }
            mma_commit(bar_dn);
        }
        RM_STAMP(12);
    };

    // ---- phase: add this CTA's [T x Hs] partial of y to the residual stream
    // The last flush of a run (no loads are in flight into the gate/up stage any more; the staged partial sums that
    // may have used it have been consumed, or the owners' h could not have arrived) goes through that stage: the
    // accumulator is laid out as [token][128 columns] per 128-column block, scaled by the gate, and the copy engine
    // adds each block to the output as one box of the [B, T, H] tensor map.  Earlier flushes of a run (batches) and
    // the anchor step, which also accumulates the ungated partial into y_anchor, add with red.global from registers.
    bool bulk_pending = false;
    auto flush = [&](const TileRef& tr, bool final_tile) {
        if (final_tile && anchor_mode != RM_ANCHOR_WRITE) {
            float* stage = reinterpret_cast<float*>(gbase + S::OFF_GU);
            stage_partial<NTOK, HS>(stage, gate ? gate + (size_t)tr.b * H : nullptr, tmem_d2, warp & 3, lane, (warp >> 2) * 32,
                                    64, T, j * HS);
            tc_fence_before();
            fence_proxy_async_smem();
            __syncthreads();
            if (tid == 0) {
#pragma unroll
                for (int mm = 0; mm < HS / 128; ++mm)
                    tensor_reduce_add_3d(&tmOut, j * HS + mm * 128, 0, tr.b, smem_u32(stage + mm * NTOK * 128));
                bulk_commit();
                bulk_pending = true;
            }
            RM_STAMP(14);
            return;
        }
        flush_partial<NTOK, HS>(a.r_out + (size_t)tr.b * T * H, a.y_anchor ? a.y_anchor + (size_t)tr.b * T * H : nullptr,
                                gate ? gate + (size_t)tr.b * H : nullptr, anchor_mode == RM_ANCHOR_WRITE, tmem_d2,
                                warp & 3, lane, (warp >> 2) * 32, 64, T, H, j * HS);
        tc_fence_before();
        __syncthreads();
        RM_STAMP(14);
    };

    // ---- duties shared by all CTAs (any time after the dependency wait).  Episodes without a single active neuron have
    // no cluster working on them: their residual passes through here.  Then the buffer the next layer accumulates
    // into is cleared.  CTAs with tiles do this while they wait for the first tile's partial sums, so that it is not
    // the tail of the kernel (the next layer's dependency wait ends when the last CTA exits).
    bool duties_done = false;
    auto shared_duties = [&]() {
        duties_done = true;
        if (a.add_residual) {
            for (int b = 0; b < a.B; ++b) {
                if (gPref[b + 1] != gPref[b]) continue;
                const float4* src = reinterpret_cast<const float4*>(a.r_in + (size_t)b * T * H);
                float* dst = a.r_out + (size_t)b * T * H;
                for (size_t i = (size_t)blockIdx.x * FT + tid; i < (size_t)T * H / 4; i += (size_t)gridDim.x * FT) {
                    const float4 v = src[i];
                    add_residual4(ya_update, gate, H, dst + 4 * i, (size_t)b * T * H + (4 * i / H) * H, (int)(4 * i % H), b, v.x, v.y, v.z, v.w);
                }
            }
        }
        if (a.zero_buf) {
            const size_t n4 = (size_t)a.B * T * H / 4;
            float4* z = reinterpret_cast<float4*>(a.zero_buf);
            for (size_t i = (size_t)blockIdx.x * FT + tid; i < n4; i += (size_t)gridDim.x * FT)
                z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };

    if (!PIPE) {
        // ---- one tile at a time: open, gate/up, scatter, owner work, down.  Loads of the next tile are issued as
        // soon as the stage they go to is free, so they travel during the exchanges.
        for (int i = 0; i < n_tiles; ++i) {
            const TileRef tr = tile_ref(g_lo + i);
            open_tile(i);
            cp_async_wait<0>();            // this tile's gate/up and down rows have landed
            fence_proxy_async_smem();
            __syncthreads();
            RM_STAMP(6);
            float ha_pre[TPL];
            anchor_prefetch(i, tr, ha_pre);
            mma_gu(i);
            wait_bar(bar_gu(0), phase_of(i));
            tc_fence_after();
            RM_STAMP(7);
            const bool refill = i + 1 < n_tiles;
            if (refill) issue_gu(g_lo + i + 1);
            cp_async_commit();
            scatter(i, refill);
            if (i == 0) shared_duties();
            wait_bar(bar_p(0), phase_of(i));           // every source's partial sums for this CTA's neurons are here
            RM_STAMP(9);
            reduce_bcast(i, tr, ha_pre);
            wait_bar(bar_h(0), phase_of(i));           // h of the whole tile (all 8 owners' atoms) is here
            RM_STAMP(11);
            mma_dn(i, tr);
            wait_bar(bar_dn, par_dn);                  // the down stage and the h tiles may be reused
            par_dn ^= 1;
            tc_fence_after();
            if (refill) issue_dn(g_lo + i + 1);
            cp_async_commit();
            RM_STAMP(13);
            if (tr.last) flush(tr, !refill);
#ifdef RM_PHASE_TIMING
            stamp_ok = false;              // first tile only
#endif
        }
    } else if (n_tiles > 0) {
        // ---- two tiles in flight: the gate/up product and the scatter of tile i+1 are issued before the owner work
        // and the down projection of tile i, so each exchange travels while the other tile's work runs.
        open_tile(0);
        cp_async_wait<0>();
        fence_proxy_async_smem();
        __syncthreads();
        RM_STAMP(6);
        mma_gu(0);
        wait_bar(bar_gu(0), 0);
        tc_fence_after();
        RM_STAMP(7);
        if (1 < n_tiles) issue_gu(g_lo + 1);
        cp_async_commit();
        scatter(0, 1 < n_tiles);
        for (int i = 0; i < n_tiles; ++i) {
            const TileRef tr = tile_ref(g_lo + i);
            const bool more = i + 1 < n_tiles;
            if (more) {
                open_tile(i + 1);
                if (i == 0) cp_async_wait<0>(); else cp_async_wait<1>();      // gate/up rows of tile i+1 have landed
                fence_proxy_async_smem();
                __syncthreads();
                mma_gu(i + 1);
            }
            float ha_pre[TPL];
            anchor_prefetch(i, tr, ha_pre);
            wait_bar(bar_p(buf_of(i)), phase_of(i));
            RM_STAMP(9);
            reduce_bcast(i, tr, ha_pre);
            if (more) {
                wait_bar(bar_gu(buf_of(i + 1)), phase_of(i + 1));
                tc_fence_after();
                const bool refill = i + 2 < n_tiles;
                if (refill) issue_gu(g_lo + i + 2);
                cp_async_commit();
                // The staging area (and, without one, the gate/up stage of a last tile) is shared by consecutive
                // tiles: this CTA's copies of tile i's partial sums must all have been read before tile i+1 is staged
                // over them.  They have once h(i) is complete here: every owner has then finished its reduction.
                if (S::STAGED || !refill) wait_bar(bar_h(buf_of(i)), phase_of(i));
                scatter(i + 1, refill);
            } else {
                cp_async_commit();
            }
            wait_bar(bar_h(buf_of(i)), phase_of(i));
            RM_STAMP(11);
            cp_async_wait<1>();            // down rows of tile i have landed
            fence_proxy_async_smem();
            __syncthreads();
            mma_dn(i, tr);
            wait_bar(bar_dn, par_dn);
            par_dn ^= 1;
            tc_fence_after();
            if (more) issue_dn(g_lo + i + 1);
            cp_async_commit();
            RM_STAMP(13);
            if (tr.last) flush(tr, !more);
#ifdef RM_PHASE_TIMING
            stamp_ok = false;
#endif
        }
    }
#ifdef RM_PHASE_TIMING
    stamp_ok = true;
#endif

    // ---- teardown.  Everything peers send into this CTA's shared memory is counted on barriers this CTA has waited
    // for, so nothing is in flight towards it any more and it may exit without a cluster-wide wait.
    if (!duties_done) shared_duties();
    cp_async_wait<0>();
    if (bulk_pending) bulk_wait_read_all();        // the copy engine has read the staged accumulator
    tc_fence_before();
    if (__syncthreads_or(gave_up)) linger_after_timeout();
    if (warp == 0) tmem_dealloc(tmem_d1, S::TMEM_COLS);
    RM_STAMP(15);
    RM_WALL(3);
}

// ===============================================================================================================
// Warp-specialised variant for launches in which a cluster walks many tiles (large K, dense passes, batches).
// The same decomposition and exchanges as above, but the phases of consecutive tiles run concurrently on different
// warps, connected by mbarriers:
//   warps 0-3  scatter : wait for the gate/up product of tile i, read it from tensor memory, send the partial sums
//                        to their owners; at the end of an episode, add the down accumulator to the residual stream
//   warps 4-7  owner   : wait for the 8 partial sums of tile i, GeLU-tanh(g)*u, record, h atom, all-gather
//   warp  8    mma     : one thread issues the gate/up products of tile i, one K half at a time as the rows land
//   warps 9-10 loader  : cp.async gathers of the next tile's gate/up rows (warp 9) and down rows (warp 10) as soon
//                        as the stage (half) they go to is free
//   warp  11   mma     : one thread issues the down product of tile i as soon as h(i) is complete in this CTA
// Exchange state (D1 in tensor memory, partial-sum buffer, h tiles, h atom, staging) is double-buffered by tile
// parity.  An episode change drains the pipeline (CTA-wide barrier), prepares the new x slice and restarts.
constexpr int WT = 384;            // threads per CTA of the warp-specialised kernel (12 warps)

template <int NTOK, int HS>
struct SmemWS {
    static constexpr int KB = HS / 64;
    static constexpr bool STAGED = HS == 128;                // room for staging buffers only at H = 1024
    static constexpr int X_BYTES = KB * NTOK * 128;
    static constexpr int GU_STAGE = KB * 128 * 128;
    static constexpr int DN_STAGE = KB * NT * 128;
    static constexpr int HT_HALF = NT * 128;
    static constexpr int OFF_X = 0;
    static constexpr int OFF_GU = OFF_X + X_BYTES;
    static constexpr int OFF_DN = OFF_GU + GU_STAGE;
    static constexpr int OFF_HT = OFF_DN + DN_STAGE;         // [2 buffers][hi, lo]
    static constexpr int OFF_HS = OFF_HT + 4 * HT_HALF;      // [2 buffers] h atom (1 KB hi, 1 KB lo)
    static constexpr int OFF_SS = OFF_HS + 2 * 2048;
    static constexpr int OFF_N = OFF_SS + CS * 64 * 4;
    static constexpr int OFF_PREF = OFF_N + 8 * NT * 4;     // neuron ids of eight consecutive tiles: the loader may run up
                                                            // to six tiles ahead of the owner warps that read them
    static constexpr int OFF_BAR = ((OFF_PREF + (2 * MAXB + 1) * 4 + 7) / 8) * 8;
    static constexpr int OFF_P = ((OFF_BAR + 224 + 15) / 16) * 16;  // [2][CS][16][p_row] (+ [2] staging), sized at launch
    static constexpr int TMEM_COLS = 2 * NTOK + (HS / 128) * d2_width(NTOK, HS) <= 256 ? 256 : 512;   // D1 x 2 + D2 blocks
    static int total_bytes(int T) { return OFF_P + (STAGED ? 4 : 2) * CS * 16 * p_row_for(T) * 4 + 1024; }
};

template <int NTOK, int HS, bool EQ4>
__global__ void __launch_bounds__(WT, 1) fused_layer_ws_kernel(const FusedArgs a, const __grid_constant__ CUtensorMap tmOut) {
    const int anchor_mode = EQ4 ? a.anchor_mode : (int)RM_ANCHOR_NONE;
    const float* const gate = EQ4 ? a.gate : nullptr;
    const float* const ya_update = anchor_mode == RM_ANCHOR_UPDATE ? a.y_anchor : nullptr;
    using S = SmemWS<NTOK, HS>;
    constexpr int KB = S::KB;
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* gbase = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t sX = base + S::OFF_X, sGU = base + S::OFF_GU, sDN = base + S::OFF_DN, sHT = base + S::OFF_HT;
    const uint32_t sP = base + S::OFF_P, sSS = base + S::OFF_SS;
    const float* gSS = reinterpret_cast<const float*>(gbase + S::OFF_SS);
    int* gN = reinterpret_cast<int*>(gbase + S::OFF_N);
    int* gPref = reinterpret_cast<int*>(gbase + S::OFF_PREF);
    int* gCnt = gPref + MAXB + 1;
    const uint32_t bar0 = base + S::OFF_BAR;
    auto bar_gu = [&](int pb) { return bar0 + 8 * pb; };           // gate/up product of a tile is complete
    auto bar_p = [&](int pb) { return bar0 + 16 + 8 * pb; };       // all partial sums for this owner have arrived
    auto bar_h = [&](int pb) { return bar0 + 32 + 8 * pb; };       // all h atoms have arrived
    auto d1_free = [&](int pb) { return bar0 + 48 + 8 * pb; };     // the scatter warps have read D1[pb]
    // down product of a tile is complete.  One barrier per tile parity: a scatter warp waits for down(it - 2) only when
    // it is about to send tile it, and by then down(it - 1) may be complete as well; on a single barrier that wait
    // would then see the parity of the phase two ahead and never return.  With two, the next phase of the barrier it
    // waits on (down(it)) cannot complete before the warp itself has sent tile it.
    auto bar_dn = [&](int pb) { return bar0 + 64 + 16 * pb; };
    const uint32_t bar_s = bar0 + 72;
    // the down stage is filled and consumed in two halves too (tile neurons 0..31 and 32..63)
    auto dnh_full = [&](int h) { return bar0 + 128 + 8 * h; };
    auto dnh_free = [&](int h) { return bar0 + 144 + 8 * h; };
    // the gate/up stage is filled and consumed in two halves of the K range, so that loading one half overlaps
    // the products of the other
    auto guh_full = [&](int h) { return bar0 + 88 + 8 * h; };      // the rows of one K half have landed
    auto guh_free = [&](int h) { return bar0 + 104 + 8 * h; };     // the products over one K half are complete
    const uint32_t s_tmem = bar0 + 120;
    volatile uint32_t* g_tmem = reinterpret_cast<volatile uint32_t*>(gbase + S::OFF_BAR + 120);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int j = (int)cluster_ctarank();
    const int cid = (int)cluster_id_x(), NC = (int)cluster_count_x();
    const int H = a.H, T = a.T, PR = a.p_row;
    const int p_bytes = CS * 16 * PR * 4;

    if (tid == 0) {
        for (int pb = 0; pb < 2; ++pb) {
            mbar_init(bar_gu(pb), 1); mbar_init(bar_p(pb), 1); mbar_init(bar_h(pb), 1); mbar_init(d1_free(pb), 4);
        }
        mbar_init(bar_dn(0), 1); mbar_init(bar_dn(1), 1);
        mbar_init(bar_s, 1);
        for (int h = 0; h < 2; ++h) { mbar_init(guh_full(h), 32); mbar_init(guh_free(h), 1); }
        for (int h = 0; h < 2; ++h) { mbar_init(dnh_full(h), 32); mbar_init(dnh_free(h), 1); }
        fence_mbar_init();
        int acc = 0;
        const int cap = (int)(a.list_cap < (int64_t)a.I ? a.list_cap : (int64_t)a.I);
        for (int b = 0; b < a.B; ++b) {
            int c = a.I;
            if (a.count) {                 // a list, or (no list) the leading `count` neurons of a compact layer
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
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem_d1 = *g_tmem;
    const uint32_t tmem_d2 = tmem_d1 + 2 * NTOK;
    pdl_launch_dependents();

    const int tiles_total = gPref[a.B];
    const int n_active = tiles_total < NC ? tiles_total : NC;
    const int g_lo = cid < n_active ? (int)((long long)cid * tiles_total / n_active) : 0;
    const int g_hi = cid < n_active ? (int)((long long)(cid + 1) * tiles_total / n_active) : 0;

    auto tile_ref = [&](int g) {
        TileRef r;
        int b = 0;
        while (gPref[b + 1] <= g) ++b;
        r.b = b;
        r.p0 = (g - gPref[b]) * NT;
        const int left = gCnt[b] - r.p0;
        r.nvalid = left < NT ? left : NT;
        r.first = (g == g_lo) || (g == gPref[b]);
        r.last = (g == g_hi - 1) || (g == gPref[b + 1] - 1);
        return r;
    };
    bool gave_up = false;
    bool bulk_pending = false;                 // thread 0: a bulk add of the staged accumulator is in flight
    auto wait_bar_at = [&](uint32_t bar, uint32_t parity, int line) {
        if (!mbar_wait(bar, parity)) {
            rm_set_status_at(a.status, RM_ERR_TIMEOUT, (line << 12) | (int)(blockIdx.x & 0xfffu));
            gave_up = true;
        }
    };

    // loaders: one warp gathers the gate and up rows (warp 9), one the down rows (warp 10), so neither waits for the
    // other's stage.  Lane l = (r, c): per instruction the warp covers 4 tile neurons x one 128-byte row segment
    // (8 lanes x 16 bytes, coalesced); the 16 groups of 4 neurons are walked in turn.  `it` is the cluster-local
    // tile sequence number.
    const int lr = lane >> 3, lc = lane & 7;
    // the 16 neuron ids this lane needs for a tile.  The raw loads are issued one tile ahead of their use (under a
    // saturated memory system a dependent 4-byte read costs microseconds); range checks happen at use time.
    auto fetch_ids = [&](int g, int (&nn)[16]) {
        const TileRef r = tile_ref(g);
#pragma unroll
        for (int grp = 0; grp < 16; ++grp) {
            const int q = grp * 4 + lr;
            nn[grp] = a.idx ? (q < r.nvalid ? __ldg(a.idx + (size_t)r.b * a.idx_stride + r.p0 + q) : -1)
                            : (q < r.nvalid ? r.p0 + q : -1);
        }
    };
    auto check_ids = [&](int g, int (&nn)[16], bool report) {
        const TileRef r = tile_ref(g);
        bool bad = false;
#pragma unroll
        for (int grp = 0; grp < 16; ++grp) {
            const int q = grp * 4 + lr;
            if (q < r.nvalid && (nn[grp] < 0 || nn[grp] >= a.I)) { bad = true; nn[grp] = -1; }
        }
        if (bad && report) rm_set_status(a.status, RM_ERR_INDEX);
    };
    // gate/up: the ids are checked and published before the stage is known to be free; the gathers go out after
    auto publish_gu = [&](int g, int it, int (&nn)[16]) {
        check_ids(g, nn, lc == 0);
        if (lc == 0) {
#pragma unroll
            for (int grp = 0; grp < 16; ++grp) gN[(it & 7) * NT + grp * 4 + lr] = nn[grp];
        }
        __threadfence_block();             // the neuron ids are read by the owner warps much later
    };
    constexpr int KH = KB / 2;                             // 64-column blocks per K half (1 at H = 1024, 2 at H = 2048)
    auto issue_gu_half = [&](int it, int h, const int (&nn)[16]) {
        if (lane == 0 && h == 0) RM_WS(it, 0);
#pragma unroll
        for (int grp = 0; grp < 16; ++grp) {
            const int q = grp * 4 + lr, n = nn[grp];
            const __nv_bfloat16* src = a.packed + (size_t)(n < 0 ? 0 : n) * 3 * H + (size_t)j * 3 * HS + lc * 8;
            const uint32_t d0 = sGU + q * 128 + ((lc ^ (q & 7)) << 4);
#pragma unroll
            for (int kk = 0; kk < KH; ++kk) {
                const int kb = h * KH + kk;
                cp_async16(d0 + kb * 16384, src + kb * 64, n >= 0);                       // gate row
                cp_async16(d0 + kb * 16384 + 64 * 128, src + HS + kb * 64, n >= 0);       // up row
            }
        }
        cp_async_arrive_noinc(guh_full(h));
    };
    // L2 prefetch of this CTA's pieces (3*Hs*2 contiguous bytes per neuron) of a tile that is still several tiles
    // away: the later gathers into shared memory then find their lines in the 126 MB L2, so the amount of weight data
    // in flight from HBM is no longer bounded by the shared-memory stages.  Two neurons per lane.
    auto prefetch_tile = [&](int g) {
        const TileRef r = tile_ref(g);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int q = lane + 32 * half;
            if (q < r.nvalid) {
                const int n = a.idx ? __ldg(a.idx + (size_t)r.b * a.idx_stride + r.p0 + q) : r.p0 + q;
                if (n >= 0 && n < a.I) prefetch_l2(a.packed + (size_t)n * 3 * H + (size_t)j * 3 * HS, 3 * HS * 2);
            }
        }
    };
    const int PD = a.l2_prefetch;                          // prefetch distance in tiles
    auto issue_dn_half = [&](int h, const int (&nn)[16]) {
#pragma unroll
        for (int g8 = 0; g8 < 8; ++g8) {
            const int grp = h * 8 + g8;
            const int q = grp * 4 + lr, n = nn[grp];
            const __nv_bfloat16* src = a.packed + (size_t)(n < 0 ? 0 : n) * 3 * H + (size_t)j * 3 * HS + 2 * HS + lc * 8;
            const uint32_t d0 = sDN + q * 128 + ((lc ^ (q & 7)) << 4);
#pragma unroll
            for (int cb = 0; cb < KB; ++cb) cp_async16(d0 + cb * 8192, src + cb * 64, n >= 0);
        }
        cp_async_arrive_noinc(dnh_full(h));
    };

    __syncthreads();                       // gPref / gCnt

    constexpr uint32_t IDESC_GU = idesc_bf16_f32(128, NTOK, false, false);
    constexpr uint32_t IDESC_DN = idesc_bf16_f32(128, d2_width(NTOK, HS), true, true);
    const uint64_t desc_k = smem_desc_sw128(0, 16, 1024);
    const uint64_t desc_mn = smem_desc_sw128(0, 8192, 1024);
    const int n_tiles = g_hi - g_lo;
    uint32_t par_s = 0;
    bool waited_prev = false;              // griddepcontrol.wait has been executed by this thread

    // ---- segments: maximal runs of this cluster's tiles within one episode
    int it0 = 0;                            // cluster-local sequence number of the segment's first tile
    while (it0 < n_tiles) {
        const TileRef tr0 = tile_ref(g_lo + it0);
        const int b = tr0.b;
        int seg = 1;
        while (it0 + seg < n_tiles && tile_ref(g_lo + it0 + seg).b == b) ++seg;

        if (warp == 9 || warp == 10) {
            // loader warps: the segment's first tile goes out before anything else (stages are free after a drain)
            int nn[16];
            fetch_ids(g_lo + it0, nn);
            if (warp == 9) { publish_gu(g_lo + it0, it0, nn); issue_gu_half(it0, 0, nn); issue_gu_half(it0, 1, nn); }
            else {
                check_ids(g_lo + it0, nn, false);
                issue_dn_half(0, nn);
                issue_dn_half(1, nn);
                for (int d = 1; d <= PD && d < seg; ++d) prefetch_tile(g_lo + it0 + d);
            }
        } else if (warp < 8) {
            // scatter and owner warps: x slice of episode b (256-thread mapping)
            constexpr int PARTS = 256 / NTOK;
            constexpr int CPP = HS / PARTS;
            const int t = tid / PARTS, part = tid % PARTS;
            int n_share = 1, my_share = 0;
            if (a.add_residual) {          // integer divisions (~0.8 us): ahead of the dependency wait
                const long long e0 = gPref[b], e1 = gPref[b + 1];
                int first_c = (int)((e0 * n_active) / tiles_total);
                while ((long long)(first_c + 1) * tiles_total / n_active <= e0) ++first_c;
                int last_c = (int)(((e1 - 1) * n_active) / tiles_total);
                while (last_c + 1 < n_active && (long long)(last_c + 1) * tiles_total / n_active < e1) ++last_c;
                n_share = last_c - first_c + 1;
                my_share = cid - first_c;
            }
            if (!waited_prev) { pdl_wait(); waited_prev = true; }
            if (a.x) {
                const uint4* src = reinterpret_cast<const uint4*>(a.x + ((size_t)b * T + t) * H + (size_t)j * HS + part * CPP);
#pragma unroll
                for (int i = 0; i < CPP / 8; ++i) {
                    const uint4 u = t < T ? src[i] : make_uint4(0, 0, 0, 0);
                    const int k = part * CPP + i * 8;
                    *reinterpret_cast<uint4*>(gbase + S::OFF_X + (k >> 6) * (NTOK * 128) + t * 128 +
                                              ((((k & 63) >> 3) ^ (t & 7)) << 4)) = u;
                }
            } else {
                float v[CPP];
                float ss = 0.f;
                if (t < T) {
                    const float4* src = reinterpret_cast<const float4*>(a.r_in + ((size_t)b * T + t) * H + (size_t)j * HS + part * CPP);
#pragma unroll
                    for (int i = 0; i < CPP / 4; ++i) {
                        const float4 f = src[i];
                        v[4 * i] = f.x; v[4 * i + 1] = f.y; v[4 * i + 2] = f.z; v[4 * i + 3] = f.w;
                    }
#pragma unroll
                    for (int i = 0; i < CPP; ++i) ss = fmaf(v[i], v[i], ss);
                } else {
#pragma unroll
                    for (int i = 0; i < CPP; ++i) v[i] = 0.f;
                }
#pragma unroll
                for (int d = 1; d < PARTS; d <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
                if (tid == 0) mbar_arrive_expect_tx(bar_s, CS * NTOK * 4);
#pragma unroll
                for (int dst = part; dst < CS; dst += PARTS)
                    st_async_f32(map_to_rank(sSS + (j * 64 + t) * 4, dst), ss, map_to_rank(bar_s, dst));
                if (a.add_residual && t < T && (t % n_share) == my_share) {
                    const size_t row = ((size_t)b * T + t) * H;
                    const int col = j * HS + part * CPP;
#pragma unroll
                    for (int i = 0; i < CPP / 4; ++i)
                        add_residual4(ya_update, gate, H, a.r_out + row + col + 4 * i, row, col + 4 * i, b, v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                }
                wait_bar(bar_s, par_s);
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
            fence_proxy_async_smem();
        }
        if (!a.x) par_s ^= 1;
        __syncthreads();                   // x is in place for the mma warp

        if (warp < 4) {
            // ================= scatter warps
            for (int k = 0; k < seg; ++k) {
                const int it = it0 + k, pb = it & 1;
                wait_bar(bar_gu(pb), (it >> 1) & 1);
                tc_fence_after();
                if (tid == 0) RM_WS(it, 2);
                // down(it-2) has finished reading the h tiles of this parity, and (through the chain h(it-2) <- every
                // owner's reduction) the owners are done with the exchange buffer of this parity: only now may this
                // tile's partial sums go out, because they let the owners refill both
                if (k >= 2) wait_bar(bar_dn(pb), ((it - 2) >> 1) & 1);
                const uint32_t d1 = tmem_d1 + pb * NTOK;
                const bool last_of_all = it == n_tiles - 1;
                const bool stage_in_gu = !S::STAGED && last_of_all && p_bytes <= S::GU_STAGE;
                if (S::STAGED || stage_in_gu) {
                    unsigned char* stg = S::STAGED ? gbase + S::OFF_P + (2 + pb) * p_bytes : gbase + S::OFF_GU;
                    for (int c0 = 0; c0 < NTOK; c0 += 32) {
                        float v[32];
                        const int m = warp * 32 + lane;
                        tmem_ld32(d1 + ((uint32_t)(warp * 32) << 16) + c0, v);
                        const int q = m & 63;
                        float* row = reinterpret_cast<float*>(stg) + (((q >> 3) * 16 + (m >> 6) * 8 + (q & 7)) * PR + c0);
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            if (c0 + 4 * e < PR)
                                *reinterpret_cast<float4*>(row + 4 * e) = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(d1_free(pb));
                    fence_proxy_async_smem();
                    named_barrier(2, 128);
                    if (tid < CS)
                        bulk_copy_to_peer(map_to_rank(sP + pb * p_bytes + (j * 16 * PR) * 4, tid),
                                          smem_u32(stg) + tid * 16 * PR * 4, 16 * PR * 4, map_to_rank(bar_p(pb), tid));
                } else {
                    for (int c0 = 0; c0 < NTOK; c0 += 32) {
                        float v[32];
                        const int m = warp * 32 + lane;
                        tmem_ld32(d1 + ((uint32_t)(warp * 32) << 16) + c0, v);
                        const int q = m & 63;
                        const uint32_t dst = map_to_rank(sP + pb * p_bytes + ((j * 16 + (m >> 6) * 8 + (q & 7)) * PR + c0) * 4, q >> 3);
                        const uint32_t rbar = map_to_rank(bar_p(pb), q >> 3);
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            if (c0 + 4 * e < PR) st_async_v4(dst + e * 16, v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3], rbar);
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(d1_free(pb));
                }
                if (tid == 0) RM_WS(it, 3);
            }
            // follow the remaining phases of the down barrier in order (a parity wait can only tell the current phase
            // from the previous one)
            if (seg >= 2) wait_bar(bar_dn((it0 + seg - 2) & 1), ((it0 + seg - 2) >> 1) & 1);
            // end of the episode's run: add this CTA's [T x Hs] partial of y to the residual stream
            {
                const int it = it0 + seg - 1;
                wait_bar(bar_dn(it & 1), (it >> 1) & 1);
                tc_fence_after();
                if (it == n_tiles - 1 && anchor_mode != RM_ANCHOR_WRITE) {
                    // last flush of the run: nothing is in flight into the gate/up stage any more.  The accumulator
                    // goes there as [token][128 columns] per 128-column block, scaled by the gate, and the copy
                    // engine adds each block to the output as one box of the [B, T, H] tensor map.
                    float* stage = reinterpret_cast<float*>(gbase + S::OFF_GU);
                    stage_partial<NTOK, HS>(stage, gate ? gate + (size_t)b * H : nullptr, tmem_d2, warp, lane, 0, 32, T, j * HS);
                    tc_fence_before();
                    fence_proxy_async_smem();
                    named_barrier(2, 128);
                    if (tid == 0) {
#pragma unroll
                        for (int mm = 0; mm < HS / 128; ++mm)
                            tensor_reduce_add_3d(&tmOut, j * HS + mm * 128, 0, b, smem_u32(stage + mm * NTOK * 128));
                        bulk_commit();
                        bulk_pending = true;
                    }
                } else {
                    flush_partial<NTOK, HS>(a.r_out + (size_t)b * T * H, a.y_anchor ? a.y_anchor + (size_t)b * T * H : nullptr,
                                            gate ? gate + (size_t)b * H : nullptr, anchor_mode == RM_ANCHOR_WRITE, tmem_d2,
                                            warp, lane, 0, 32, T, H, j * HS);
                    tc_fence_before();
                }
            }
        } else if (warp < 8) {
            // ================= owner warps: warp ow handles local neurons ow and ow + 4, one per half-warp; a lane
            // owns TPL consecutive tokens of its neuron
            const int ow = warp - 4, ot = tid - 128;
            constexpr int TPL = NTOK / 16;                 // 4 tokens per lane at NTOK = 64, 2 at NTOK = 32
            const int ql = ow + 4 * (lane >> 4);
            const int t0 = (lane & 15) * TPL;
            for (int k = 0; k < seg; ++k) {
                const int it = it0 + k, pb = it & 1;
                if (ot == 0) {
                    // the bulk-copy route moves whole padded rows, the per-thread stores only the columns that exist
                    // in tensor memory (the row pad can exceed the token tile)
                    const bool bulk = S::STAGED || (it == n_tiles - 1 && p_bytes <= S::GU_STAGE);
                    mbar_arrive_expect_tx(bar_p(pb), bulk ? p_bytes : CS * 16 * (PR < NTOK ? PR : NTOK) * 4);
                }
                wait_bar(bar_p(pb), (it >> 1) & 1);
                if (ot == 0) RM_WS(it, 4);
                // Eq. 4: the anchor's h for this lane's tokens (the tile's neuron ids are known to be published only
                // now: the partial sums that just arrived were computed from rows gathered by those ids)
                float ha_pre[TPL];
#pragma unroll
                for (int e = 0; e < TPL; ++e) ha_pre[e] = 0.f;
                const int n_own = anchor_mode != RM_ANCHOR_NONE ? gN[(it & 7) * NT + j * 8 + ql] : -1;
                float* hap = (n_own >= 0 && t0 < T) ? a.h_anchor + ((size_t)b * a.I + n_own) * a.h_stride + t0 : nullptr;
                if (anchor_mode == RM_ANCHOR_UPDATE && hap) {
                    if (TPL == 4) {
                        const float4 f = *reinterpret_cast<const float4*>(hap);
                        ha_pre[0] = f.x; ha_pre[1] = f.y; ha_pre[2] = f.z; ha_pre[TPL - 1] = f.w;
                    } else {
                        const float2 f = *reinterpret_cast<const float2*>(hap);
                        ha_pre[0] = f.x; ha_pre[TPL - 1] = f.y;
                    }
#pragma unroll
                    for (int e = 0; e < TPL; ++e) if (t0 + e >= T) ha_pre[e] = 0.f;
                }

                const float* gP = reinterpret_cast<const float*>(gbase + S::OFF_P + pb * p_bytes);
                unsigned char* gHS = gbase + S::OFF_HS + pb * 2048;
                float gsum[TPL], usum[TPL];
#pragma unroll
                for (int e = 0; e < TPL; ++e) gsum[e] = usum[e] = 0.f;
                if (t0 < PR) {
#pragma unroll
                    for (int src = 0; src < CS; ++src) {
                        const float* pg = gP + (src * 16 + ql) * PR + t0;
                        const float* pu = gP + (src * 16 + 8 + ql) * PR + t0;
                        if (TPL == 4) {
                            const float4 g4 = *reinterpret_cast<const float4*>(pg), u4 = *reinterpret_cast<const float4*>(pu);
                            gsum[0] += g4.x; gsum[1] += g4.y; gsum[2] += g4.z; gsum[TPL - 1] += g4.w;
                            usum[0] += u4.x; usum[1] += u4.y; usum[2] += u4.z; usum[TPL - 1] += u4.w;
                        } else {
                            const float2 g2 = *reinterpret_cast<const float2*>(pg), u2 = *reinterpret_cast<const float2*>(pu);
                            gsum[0] += g2.x; gsum[TPL - 1] += g2.y;
                            usum[0] += u2.x; usum[TPL - 1] += u2.y;
                        }
                    }
                }
                float rec = 0.f;
                float hv[TPL];
#pragma unroll
                for (int e = 0; e < TPL; ++e) {
                    hv[e] = (t0 + e < T) ? rm_gelu_tanh(gsum[e]) * usum[e] : 0.f;
                    rec += fabsf(hv[e]);
                }
                if (hap) {
                    if (anchor_mode == RM_ANCHOR_WRITE) {
                        if (TPL == 4) *reinterpret_cast<float4*>(hap) = make_float4(hv[0], hv[1], hv[2], hv[TPL - 1]);
                        else *reinterpret_cast<float2*>(hap) = make_float2(hv[0], hv[TPL - 1]);
                    } else {
#pragma unroll
                        for (int e = 0; e < TPL; ++e) hv[e] -= ha_pre[e];
                    }
                }
                // TPL consecutive tokens of one neuron row: one 8-byte (or 4-byte) store each for hi and lo
                unsigned char* rowp = gHS + ql * 128 + ((((t0 >> 3) ^ ql) & 7) << 4) + (t0 & 7) * 2;
                {
                    const __nv_bfloat162 hi0 = __floats2bfloat162_rn(hv[0], hv[1]);
                    const float2 f0 = __bfloat1622float2(hi0);
                    const __nv_bfloat162 lo0 = __floats2bfloat162_rn(hv[0] - f0.x, hv[1] - f0.y);
                    if (TPL == 4) {
                        const __nv_bfloat162 hi1 = __floats2bfloat162_rn(hv[2], hv[TPL - 1]);
                        const float2 f1 = __bfloat1622float2(hi1);
                        const __nv_bfloat162 lo1 = __floats2bfloat162_rn(hv[2] - f1.x, hv[TPL - 1] - f1.y);
                        uint2 hw, lw;
                        hw.x = *reinterpret_cast<const uint32_t*>(&hi0); hw.y = *reinterpret_cast<const uint32_t*>(&hi1);
                        lw.x = *reinterpret_cast<const uint32_t*>(&lo0); lw.y = *reinterpret_cast<const uint32_t*>(&lo1);
                        *reinterpret_cast<uint2*>(rowp) = hw;
                        *reinterpret_cast<uint2*>(rowp + 1024) = lw;
                    } else {
                        *reinterpret_cast<__nv_bfloat162*>(rowp) = hi0;
                        *reinterpret_cast<__nv_bfloat162*>(rowp + 1024) = lo0;
                    }
                }
                if (a.record) {
#pragma unroll
                    for (int d = 8; d > 0; d >>= 1) rec += __shfl_xor_sync(0xffffffffu, rec, d);
                    const int n = gN[(it & 7) * NT + j * 8 + ql];
                    if ((lane & 15) == 0 && n >= 0)
                        a.record[(size_t)b * a.record_stride + n] = a.record_scale ? rec * a.record_scale[n] : rec;
                }
                fence_proxy_async_smem();
                named_barrier(1, 128);
                if (ot < 2 * CS) {
                    const int dst = ot >> 1, part = ot & 1;
                    bulk_copy_to_peer(map_to_rank(sHT + pb * 2 * S::HT_HALF + part * S::HT_HALF + j * 1024, dst),
                                      smem_u32(gHS) + part * 1024, 1024, map_to_rank(bar_h(pb), dst));
                }
                if (ot == 0) RM_WS(it, 5);
            }
        } else if (warp == 8) {
            // ================= gate/up issuer (one thread)
            if (lane == 0) {
                for (int k = 0; k < seg; ++k) {
                    const int it = it0 + k, pb = it & 1;
                    if (it >= 2) wait_bar(d1_free(pb), ((it - 2) >> 1) & 1);      // the scatter warps have read D1[pb]
                    // one proxy fence covers both halves when the second has landed by the time the first is seen
                    // (the fence costs 0.3-0.6 us here, and the loaders usually run ahead)
                    bool both = false;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (h == 0 || !both) {
                            wait_bar(guh_full(h), it & 1);
                            if (h == 0) both = mbar_try_wait(guh_full(1), it & 1);
                            fence_proxy_async_smem();
                        }
                        if (h == 0) RM_WS(it, 1);
                        tc_fence_after();
#pragma unroll
                        for (int kk = 0; kk < KH; ++kk)
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks) {
                                const int kb = h * KH + kk;
                                mma_bf16_ss(tmem_d1 + pb * NTOK, desc_k | desc_addr(sGU + kb * 16384 + ks * 32),
                                            desc_k | desc_addr(sX + kb * (NTOK * 128) + ks * 32), IDESC_GU, (kb | ks) != 0);
                            }
                        mma_commit(guh_free(h));
                    }
                    mma_commit(bar_gu(pb));
                }
            }
        } else if (warp == 11) {
            // ================= down issuer (one thread)
            if (lane == 0) {
                for (int k = 0; k < seg; ++k) {
                    const int it = it0 + k, pb = it & 1;
                    mbar_arrive_expect_tx(bar_h(pb), CS * 2048);
                    wait_bar(bar_h(pb), (it >> 1) & 1);
                    RM_WS(it, 6);
                    const uint32_t ht = sHT + pb * 2 * S::HT_HALF;
                    bool both = false;         // as in the gate/up issuer: one proxy fence when both halves are in
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (h == 0 || !both) {
                            wait_bar(dnh_full(h), it & 1);
                            if (h == 0) both = mbar_try_wait(dnh_full(1), it & 1);
                            fence_proxy_async_smem();
                        }
                        RM_WS(it, 8 + 2 * h);
                        tc_fence_after();
#pragma unroll
                        for (int mm = 0; mm < HS / 128; ++mm)
#pragma unroll
                            for (int k2 = 0; k2 < 2; ++k2) {
                                const int ks = h * 2 + k2;
                                const uint64_t aa = desc_mn | desc_addr(sDN + mm * 16384 + ks * 2048);
                                mma_bf16_ss(tmem_d2 + mm * d2_width(NTOK, HS), aa, desc_mn | desc_addr(ht + ks * 2048), IDESC_DN,
                                            !(k == 0 && ks == 0));
                                if (!d2_wide(NTOK, HS))
                                    mma_bf16_ss(tmem_d2 + mm * NTOK, aa, desc_mn | desc_addr(ht + S::HT_HALF + ks * 2048), IDESC_DN, true);
                            }
                        mma_commit(dnh_free(h));
                        if (h == 0) RM_WS(it, 9);
                    }
                    mma_commit(bar_dn(pb));
                    RM_WS(it, 7);
                }
            }
        } else {
            // ================= loader warps: tiles after the segment's first
            int nxt[16];
            if (seg > 1) fetch_ids(g_lo + it0 + 1, nxt);
            for (int k = 1; k < seg; ++k) {
                const int it = it0 + k;
                int nn[16];
#pragma unroll
                for (int grp = 0; grp < 16; ++grp) nn[grp] = nxt[grp];
                if (k + 1 < seg) fetch_ids(g_lo + it + 1, nxt);              // in flight while this tile is handled
                if (warp == 9) {
                    publish_gu(g_lo + it, it, nn);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        wait_bar(guh_free(h), (it - 1) & 1);                  // the previous tile is done with this half
                        issue_gu_half(it, h, nn);
                    }
                } else {
                    if (k + PD < seg) prefetch_tile(g_lo + it + PD);
                    check_ids(g_lo + it, nn, false);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        wait_bar(dnh_free(h), (it - 1) & 1);                  // the previous tile is done with this half
                        if (lane == 0) RM_WS(it, 11 + 2 * h);
                        issue_dn_half(h, nn);
                        if (lane == 0 && h == 0) RM_WS(it, 12);
                    }
                }
            }
        }
        __syncthreads();                   // drain: every role is done with this episode's run
        it0 += seg;
    }

    // ---- duties: residual of episodes without active neurons, and the buffer a later layer accumulates into
    if (warp < 8) {
        if (!waited_prev) { pdl_wait(); waited_prev = true; }
        if (a.add_residual) {
            for (int b = 0; b < a.B; ++b) {
                if (gPref[b + 1] != gPref[b]) continue;
                const float4* src = reinterpret_cast<const float4*>(a.r_in + (size_t)b * T * H);
                float* dst = a.r_out + (size_t)b * T * H;
                for (size_t i = (size_t)blockIdx.x * 256 + tid; i < (size_t)T * H / 4; i += (size_t)gridDim.x * 256) {
                    const float4 v = src[i];
                    add_residual4(ya_update, gate, H, dst + 4 * i, (size_t)b * T * H + (4 * i / H) * H, (int)(4 * i % H), b, v.x, v.y, v.z, v.w);
                }
            }
        }
        if (a.zero_buf) {
            const size_t n4 = (size_t)a.B * T * H / 4;
            float4* z = reinterpret_cast<float4*>(a.zero_buf);
            for (size_t i = (size_t)blockIdx.x * 256 + tid; i < n4; i += (size_t)gridDim.x * 256)
                z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
    cp_async_wait<0>();
    if (bulk_pending) bulk_wait_read_all();        // the copy engine has read the staged accumulator
    tc_fence_before();
    if (__syncthreads_or(gave_up)) linger_after_timeout();
    if (warp == 8) tmem_dealloc(tmem_d1, S::TMEM_COLS);
}

template <int NTOK, int HS>
int launch_fused_ws(rm_ctx* ctx, const FusedArgs& a, int n_clusters, bool pdl, cudaStream_t s) {
    using S = SmemWS<NTOK, HS>;
    const bool eq4 = a.anchor_mode != RM_ANCHOR_NONE || a.gate != nullptr;
    auto kern = eq4 ? fused_layer_ws_kernel<NTOK, HS, true> : fused_layer_ws_kernel<NTOK, HS, false>;
    const int smem = S::total_bytes(a.T);
    static rm_smem_configured configured = {};
    if (!configured.covers(ctx->device, smem)) {
        RM_CUDA_TRY(cudaFuncSetAttribute(fused_layer_ws_kernel<NTOK, HS, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        RM_CUDA_TRY(cudaFuncSetAttribute(fused_layer_ws_kernel<NTOK, HS, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        configured.set(ctx->device, smem);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_clusters * CS);
    cfg.blockDim = dim3(WT);
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
    alignas(64) CUtensorMap tm_out;
    const int rc = rm_make_out_map(&tm_out, a.r_out, a.B, a.T, a.H, NTOK);
    if (rc != RM_OK) return rc;
    RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, a, tm_out));
    ctx->launches++;
    return RM_OK;
}

template <int NTOK, int HS, bool PIPE>
int launch_fused(rm_ctx* ctx, const FusedArgs& a, int n_clusters, bool pdl, cudaStream_t s) {
    using S = Smem<NTOK, HS, PIPE>;
    const bool eq4 = a.anchor_mode != RM_ANCHOR_NONE || a.gate != nullptr;
    auto kern = eq4 ? fused_layer_kernel<NTOK, HS, PIPE, true> : fused_layer_kernel<NTOK, HS, PIPE, false>;
    const int smem = S::total_bytes(a.T);
    static rm_smem_configured configured = {};
    if (!configured.covers(ctx->device, smem)) {
        RM_CUDA_TRY(cudaFuncSetAttribute(fused_layer_kernel<NTOK, HS, PIPE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        RM_CUDA_TRY(cudaFuncSetAttribute(fused_layer_kernel<NTOK, HS, PIPE, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        configured.set(ctx->device, smem);
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
    alignas(64) CUtensorMap tm_out;
    const int rc = rm_make_out_map(&tm_out, a.r_out, a.B, a.T, a.H, NTOK);
    if (rc != RM_OK) return rc;
    RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, a, tm_out));
    ctx->launches++;
    return RM_OK;
}

template <int NTOK, int HS, bool PIPE>
int max_clusters(int T, int* out) {
    using S = Smem<NTOK, HS, PIPE>;
    auto kern = fused_layer_kernel<NTOK, HS, PIPE, false>;
    const int smem = S::total_bytes(T);
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
    return RM_OK;
}

}  // namespace

int rm_fused_debug_stamps(long long* host_out, int n) {
#ifdef RM_PHASE_TIMING
    if (n == -(16 * 16 * 16))
        return cudaMemcpyFromSymbol(host_out, g_ws_stamps, sizeof(long long) * 16 * 16 * 16) == cudaSuccess ? RM_OK : RM_ERR_CUDA;
    if (n < 0) {                           // negative n: the wall-clock stamps, -n values
        n = -n;
        if (n > 64 * 256 * 4) n = 64 * 256 * 4;
        return cudaMemcpyFromSymbol(host_out, g_wall_stamps, sizeof(long long) * n) == cudaSuccess ? RM_OK : RM_ERR_CUDA;
    }
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
    // The occupancy query counts one CTA per SM for kernels that allocate tensor memory; clusters beyond that
    // number simply queue, so it is a sizing hint, not a limit.
    ctx->fused_clusters = 0;
    ctx->fused_blocks_per_sm = 1;
    int n = 0, rc = RM_OK;
    if (ctx->g.H == 1024) rc = max_clusters<64, 128, false>(64, &n);
    else if (ctx->g.H == 2048) rc = max_clusters<64, 256, false>(64, &n);
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
    a.p_row = p_row_for(la.T);
    a.add_residual = add_residual ? 1 : 0;
    a.status = ctx->d_status;
    a.wall_seq = (int)(ctx->launches & 63);
    a.l2_prefetch = ctx->l2_prefetch;
    a.anchor_mode = la.anchor_mode;
    a.y_anchor = la.y_anchor;
    a.h_anchor = la.h_anchor;
    a.h_stride = la.h_stride;
    a.gate = la.gate;
    // Tiles of 64 neurons in this launch, when the host knows the number of active neurons (dense calls, or the
    // caller's hint); 0 = unknown.
    const int per_episode = la.count ? rm_effective_count_hint(ctx) : ctx->g.I;
    const long long tiles = per_episode > 0 ? (long long)((per_episode + NT - 1) / NT) * la.B : 0;
    // Variant.  H = 1024: the lean kernel for every launch (112 KB and 107 registers: two CTAs per SM, so a cluster's
    // exchange waits are covered by its SM-mate and consecutive layers overlap); measured, 33 of its clusters are
    // co-resident, two more than twice the number the occupancy query reports for one CTA per SM.  H = 2048 (one CTA
    // per SM either way): the lean kernel while every cluster gets a single tile, else the warp-specialised kernel,
    // which runs the phases of consecutive tiles concurrently.
    // (an SM has 228 KB of shared memory, of which every resident CTA also takes 1 KB of system space)
    const int lean_bytes = la.T <= 32 ? Smem<32, 128, false>::total_bytes(la.T) : Smem<64, 128, false>::total_bytes(la.T);
    const bool two_per_sm = ctx->g.H == 1024 && 2 * (lean_bytes + 1024) <= 228 * 1024;
    int cap = two_per_sm ? 2 * ctx->fused_clusters + 2 : ctx->fused_clusters;
    if (ctx->max_clusters_override > 0) cap = ctx->max_clusters_override;
    int variant = ctx->variant_override == 5 ? 0 : ctx->variant_override;    // 5: a call the whole-step kernel does not cover
    if (variant == 0) variant = (ctx->g.H == 1024 || (tiles > 0 && tiles <= cap)) ? 1 : 3;
    if (variant == 3) {
        const int fits_t = ctx->g.H == 1024 ? SmemWS<64, 128>::total_bytes(la.T) : SmemWS<64, 256>::total_bytes(la.T);
        if (fits_t > 232448) variant = 2;
        else if (ctx->max_clusters_override <= 0 || cap > ctx->fused_clusters) cap = ctx->fused_clusters;
    }
    if (variant == 2 && ctx->max_clusters_override <= 0) cap = ctx->fused_clusters;      // one CTA per SM
    // Clusters: no more than the cap, and when the tile count is known, the fewest that keep the longest run of
    // tiles per cluster as short as the cap allows (40 tiles under a cap of 32: 20 clusters of 2, not 32 of 1 or 2).
    // (The warp-specialised kernel streams, and is faster with every co-resident cluster pulling on the memory.)
    int nc = cap;
    if (tiles > 0) {
        const long long run = (tiles + cap - 1) / cap;
        nc = variant == 3 ? (int)(tiles < cap ? tiles : cap) : (int)((tiles + run - 1) / run);
    }
    const bool small_t = la.T <= 32;
    ctx->last_variant = variant;
    if (variant == 3) {
        if (ctx->g.H == 1024)
            return small_t ? launch_fused_ws<32, 128>(ctx, a, nc, pdl, s) : launch_fused_ws<64, 128>(ctx, a, nc, pdl, s);
        return small_t ? launch_fused_ws<32, 256>(ctx, a, nc, pdl, s) : launch_fused_ws<64, 256>(ctx, a, nc, pdl, s);
    }
    const bool pipe = variant == 2;
    if (ctx->g.H == 1024) {
        if (pipe)
            return small_t ? launch_fused<32, 128, true>(ctx, a, nc, pdl, s) : launch_fused<64, 128, true>(ctx, a, nc, pdl, s);
        return small_t ? launch_fused<32, 128, false>(ctx, a, nc, pdl, s) : launch_fused<64, 128, false>(ctx, a, nc, pdl, s);
    }
    // H = 2048: the two-tile variant when its buffers fit the 227 KB of an SM (they do up to T = 60), else serial
    const bool fits = Smem<64, 256, true>::total_bytes(la.T) <= 232448;
    if (small_t)
        return pipe ? launch_fused<32, 256, true>(ctx, a, nc, pdl, s) : launch_fused<32, 256, false>(ctx, a, nc, pdl, s);
    return (pipe && fits) ? launch_fused<64, 256, true>(ctx, a, nc, pdl, s) : launch_fused<64, 256, false>(ctx, a, nc, pdl, s);
}
