// Whole-step kernel of the masked gated MLP stack: ONE launch runs every layer of a denoising step.
//
// The mask of every layer is known before the step starts (it comes from an earlier, similar execution), so every
// weight address of the step is known too: loader warps stream the step's weight rows through a shared-memory ring
// without ever waiting for a layer boundary, and only the arithmetic follows the layer-to-layer dependency.
//
// Grid: clusters of 8 CTAs, all co-resident (one CTA per SM).  Per layer and episode (an "item") the active list is
// cut evenly over the clusters; a cluster walks its run in tiles of up to 256 neurons.  Inside a tile
//   gate/up : CTA j takes up to 32 of the tile's neurons and computes their gate and up rows against the whole
//             width H -- A = the neurons' weight rows (gate and up interleaved, K-major, 128-byte swizzle, gathered by
//             16-byte cp.async), B = x (64 token rows).  One tcgen05.mma costs the same ~64 clocks whatever its
//             shape up to 128 x 128, so an instruction carries two 16-column steps at once, one from each half of
//             H: A = [rows over columns of the first half ; the same rows over columns of the second half]
//             (M = 128), B = [x columns of the first half ; of the second half] (N = 128); the two diagonal
//             64 x 64 blocks of D1 are the two halves' partial sums (the off-diagonal blocks are ignored) and are
//             added in the epilogue.  No partial sums cross CTAs.
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
// The EQ4 instantiation adds the anchor-relative update (Eq. 4) and the output gate: the anchor step retains h per neuron
// and the ungated sums y_a; an update step multiplies the down rows with h - h_a and adds gate * y_a.
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
constexpr int X_BYTES = NTOK * 128;    // one 64-column block of x: 64 token rows x 128 bytes
constexpr int XSB = 2 * X_BYTES;       // x ring stage: the blocks of columns c and c + H/2
constexpr int XS_MAX = 8;
constexpr int SB = 16384;              // weight ring stage: 128 rows x 128 bytes
constexpr int EXCH = 16384;            // second-half partial sums of a tile on their way to the threads that finish them
constexpr int MAXL = 64, MAXB = 16, MAX_ITEMS = 512;   // layers, episodes, layers x episodes of one launch
constexpr int NXW = 4;                 // warps that issue the x copies (copies of one issuing thread do not overlap much)
constexpr int NTHREADS = 608;          // warps: 0-7 epilogue and normalisation, 8-11 loaders, 12 issuer, 13-16 x copies, 17 L2 prefetch,
                                       // 18 stage watcher
constexpr int W_LOAD0 = 8, W_MMA = 12, W_X0 = 13, W_PF = 17, W_WATCH = 18;
constexpr int SYNC_ABORT = MAXB;       // sync[0..MAXB): per-episode arrival counters; sync[MAXB]: abort flag
constexpr int SYNC_COPY = 32;          // sync[32..32+MAXB): per-episode counters of the CTAs that have copied r_in into r
constexpr int SYNC_READ = 48;          // sync[48..48+MAXB): per-episode counters of the CTAs that have read r for a layer's normalisation
constexpr int SYNC_ITEM = 64;          // sync[64..64+MAX_ITEMS): batches count the arrivals of every (layer, episode) by itself
constexpr int SYNC_RITEM = SYNC_ITEM + MAX_ITEMS;      // ... and the CTAs that have read the item's input rows
constexpr int SYNC_BYTES = (SYNC_RITEM + MAX_ITEMS) * 4;

struct PArgs {
    const __nv_bfloat16* packed[MAXL];
    float* r;                          // [B,T,H] fp32: r_L on exit; the layers add into it in place
    const float* r_in;                 // [B,T,H] fp32: r_0.  When it is another buffer than r, the kernel starts r as a copy of it
    __nv_bfloat16* xbuf;               // [clusters][2][H/64][64 rows x 128 bytes]: the clusters' own copies of x, stored as
                                       // the shared-memory image of each 64-column block (128-byte swizzle)
    const int32_t* idx;                // list (b, l) at idx + b * idx_b_stride + l * idx_l_stride; NULL: positions
    const int32_t* count;              // count (b, l) at count[b * count_b_stride + l]; NULL: every neuron
    int64_t idx_b_stride, idx_l_stride, list_cap, count_b_stride;
    float* record;                     // record (b, l, n) at record[b * rec_b_stride + l * I + n]; NULL: none
    int64_t rec_b_stride;
    const float* record_scale;         // [L, I] or NULL
    int* sync;                         // [0..MAXB): per-episode arrival counters, never reset between launches; [MAXB]: abort flag
    int sync_base[MAXB];               // value of each counter when this launch starts (the host keeps count)
    int copy_base[MAXB];               // the same for the copy counters
    int* status;
    int L, B, T, I;
    int per_item;                      // arrivals are counted per (layer, episode) on counters cleared before the launch (batches:
                                       // a cluster that takes no part in an episode runs ahead of those that do, so one
                                       // counter per episode could not tell the layers apart); else per episode, never cleared
    int x_ext;                         // layer 0 takes x from the caller's buffer (single-layer entry): no normalisation
    int pf_bytes;                      // weight bytes a CTA may have asked into L2 ahead of its loaders (0: no prefetch)
    // Anchor-relative update (Eq. 4) and output gate; read by the EQ4 instantiation only
    int anchor_mode;                   // RM_ANCHOR_NONE / _WRITE / _UPDATE
    float* y_anchor;                   // [L,B,T,H] fp32, pre-gate: accumulated (from zeros) in a write step, read in an update step
    float* h_anchor;                   // [L,B,I,h_stride] fp32, neuron-major: written in a write step, read in an update step
    int64_t h_stride;
    const float* gate;                 // [L,B,H] fp32 or NULL (= 1)
};

#ifdef RM_PHASE_TIMING
__device__ long long g_ps_stamps[64 * 128 * 32];
__device__ __forceinline__ long long ps_now() {
    long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define RM_PS(item, slot) do { if ((item) < 64 && blockIdx.x < 128) g_ps_stamps[((item) * 128 + blockIdx.x) * 32 + (slot)] = ps_now(); } while (0)
#define RM_PC(item, slot, v) do { if ((item) < 64 && blockIdx.x < 128) g_ps_stamps[((item) * 128 + blockIdx.x) * 32 + (slot)] = (v); } while (0)
// -DRM_PHASE_TIMING=1: the phase stamps only (a handful per layer); =2 adds clock deltas around every wait and the
// per-stage clocks of one item's gate/up stream (row 32 + who of the stamp array, one value per ring stage)
#if RM_PHASE_TIMING + 0 >= 2
#define RM_CLK() clock64()
#define RM_TRACE_ITEM 5
#define RM_TR(item, who, stage) do { if ((item) == RM_TRACE_ITEM && (stage) < 32) RM_PC(32 + (who), (stage), clock64()); } while (0)
#else
#define RM_CLK() 0ll
#define RM_TR(item, who, stage) do { } while (0)
#endif
#else
#define RM_PS(item, slot) do { } while (0)
#define RM_PC(item, slot, v) do { } while (0)
#define RM_CLK() 0ll
#define RM_TR(item, who, stage) do { } while (0)
#endif

__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_acquire_cta(const int* p) {          // shared memory
    int v;
    asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}
// The issuer's read of the landed-stage count: a relaxed load.  An acquire load holds back the product instructions
// behind it for ~160 clocks; here the order is kept by the branch on the value, by tcgen05.fence::after_thread_sync
// before the products, and by the watcher's proxy fence before its release store.
__device__ __forceinline__ int ld_relaxed_cta(const int* p) {          // shared memory
    int v;
    asm volatile("ld.relaxed.cta.shared::cta.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}
// The issuer's wait for more landed stages, kept out of line so that the loop that issues the products holds no wait
// loop: returns the count once it exceeds `stage`, or what it last read when the bounded wait ran out or the CTA aborts.
__device__ __noinline__ uint32_t landed_stages(const int* count, uint32_t stage, const int* abort_flag) {
    uint32_t ready = 0;
    for (uint32_t i = 0; i < (1u << 24); ++i) {
        ready = (uint32_t)ld_relaxed_cta(count);
        if (stage < ready) break;
        if ((i & 4095u) == 4095u && *reinterpret_cast<const volatile int*>(abort_flag)) break;
    }
    return ready;
}
__device__ __noinline__ void report_timeout(int* status, volatile int* abort_flag, int* sync, int line) {
    rm_set_status_at(status, RM_ERR_TIMEOUT, (line << 12) | (int)(blockIdx.x & 0xfffu));
    *abort_flag = 1;
    atomicExch(sync + SYNC_ABORT, 1);
}
// The part of a bounded wait that runs when the phase was not complete at the first look.  Returns true when the waiter
// has to give up: the wait ran out (status RM_ERR_TIMEOUT with the wait's source line and the CTA), or this CTA or the
// grid is aborting.
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, int line, volatile int* abort_flag, int* sync, int* status) {
    for (uint32_t i = 0; i < (1u << 22); ++i) {
        if (mbar_try_wait(bar, parity)) return false;
        if (i > 64) __nanosleep(32);
        if ((i & 1023u) == 1023u && (*abort_flag || ((i & 16383u) == 16383u && ld_acquire_gpu(sync + SYNC_ABORT)))) {
            *abort_flag = 1;
            return true;
        }
    }
    report_timeout(status, abort_flag, sync, line);
    return true;
}
// A bounded wait for a counter in global memory, out of line (for the path that is rarely taken).  Returns true when
// the waiter has to give up.
__device__ __noinline__ bool counter_wait_slow(const int* counter, int target, int line, volatile int* abort_flag, int* sync, int* status) {
    for (uint32_t i = 0; i < (1u << 21); ++i) {
        if (ld_acquire_gpu(counter) >= target) return false;
        if ((i & 255u) == 255u && (*abort_flag || ld_acquire_gpu(sync + SYNC_ABORT))) { *abort_flag = 1; return true; }
    }
    report_timeout(status, abort_flag, sync, line);
    return true;
}
__device__ __forceinline__ void st_release_cta(int* p, int v) {         // shared memory
    asm volatile("st.release.cta.shared::cta.s32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
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
// The lists of a layer's episodes, laid end to end, are cut evenly over the clusters: cluster c takes positions
// [S c / NC, S (c + 1) / NC) of the S = sum of the counts.  Its run in episode b's list (which starts at position P
// of the concatenation and holds K neurons) is the overlap.  One episode: its list is cut evenly over all clusters.
// Several episodes: every cluster gets the same number of neurons per layer, from one or two episodes.
__device__ __forceinline__ Run cluster_run(int K, int P, int S, int c, int NC) {
    Run r;
    const int lo = (int)((long long)S * c / NC), hi = (int)((long long)S * (c + 1) / NC);
    const int a = lo > P ? lo : P, b = hi < P + K ? hi : P + K;
    r.start = a - P;
    r.n = b > a ? b - a : 0;
    r.ntiles = (r.n + CT - 1) / CT;
    return r;
}
__device__ __forceinline__ void tile_span(const Run& r, int i, int& t0, int& ts) {
    if (r.ntiles == 1) { t0 = r.start; ts = r.n; return; }
    const int a = r.n * i / r.ntiles, b = r.n * (i + 1) / r.ntiles;               // (n <= I < 2^24, i < 2^7: no overflow)
    t0 = r.start + a;
    ts = b - a;                                                    // <= 256
}
__device__ __forceinline__ void cta_span(int ts, int j, int& off, int& nj) {
    off = ts * j / CS;
    nj = ts * (j + 1) / CS - off;                                  // <= 32
}

// Down stages of a tile are taken in an order that follows the arrival of the h pieces.  CTA p sends its piece to
// p + 1, p + 2, ... in turn, so CTA j receives the pieces j - 1, j - 2, ..., j + 1 in that order (ranks mod 8, ~0.13 us
// apart); it starts with the highest stage that lies entirely below the end of its own piece (that stage needs its own
// piece and the one or two below it) and goes downwards, wrapping round, so that the stage that reaches into piece
// j + 1 comes last.  Stage number k of that order:
__device__ __forceinline__ int d_stage_first(int ts, int j, int sps, int nst) {
    const int end = ts * (j + 1) / CS;                             // end of CTA j's piece
    int s0 = end / sps - 1;
    if (s0 >= nst) s0 = nst - 1;
    return s0 < 0 ? nst - 1 : s0;
}
__device__ __forceinline__ int d_stage(int s0, int k, int nst) {
    const int s = s0 - k;
    return s < 0 ? s + nst : s;
}
// The pieces whose slots a stage reads, as a bit mask over the CTA ranks
__device__ __forceinline__ uint32_t d_stage_pieces(int ts, int s, int sps) {
    const int lo = s * sps, hi = (s + 1) * sps < ts ? (s + 1) * sps : ts;
    uint32_t m = 0;
#pragma unroll
    for (int p = 0; p < CS; ++p) {
        const int a = ts * p / CS, b = ts * (p + 1) / CS;
        if (a < hi && b > lo) m |= 1u << p;
    }
    return m;
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
struct Env { const int* sRunStart; const int* sRunN; int L, B, c, NC, x_ext, serial; };   // this cluster's run in every item's list,
                                                                                  // worked out once at the start of the kernel
__device__ __forceinline__ Run item_run(const Env& e, int item) {
    Run r;
    r.start = e.sRunStart[item];
    r.n = e.sRunN[item];
    r.ntiles = (r.n + CT - 1) / CT;
    return r;
}
__device__ __forceinline__ bool item_ext(const Env& e, int l) { return e.x_ext && l == 0; }
__device__ __forceinline__ void cur_seek(Cur& k, const Env& e) {      // to the first non-empty item at or after k.item
    const int n_items = e.L * e.B;
    while (k.item < n_items) {
        k.l = k.item / e.B;
        k.b = k.item - k.l * e.B;
        k.run = item_run(e, k.item);
        if (k.run.ntiles > 0) { k.valid = true; k.i = 0; return; }
        ++k.item;
    }
    k.valid = false;
}
__device__ __forceinline__ void cur_init(Cur& k, const Env& e) {
    k.item = 0; k.seq = 0; k.ni = 0; k.use = 0; k.i = 0;
    cur_seek(k, e);
}
// The gate/up products of tile g may be issued before the down products of tile d (the tile in front of it) when g
// does not need d's result: the same item, or an item fewer than B places further on in the (layer, episode) order --
// that is another episode, and the layer of that episode that it depends on lies before d's item.  (An item B or more
// places on can be the next layer of d's own episode, or depend on an item this cluster has not finished yet: with empty
// lists, or clusters that take no part in some episodes, the next non-empty item can be that far away.)  The epilogue
// warps prepare the input x of the next item one item ahead under exactly the same rule.
__device__ __forceinline__ bool item_may_run_ahead(int g_item, int d_item, int B) { return g_item == d_item || g_item < d_item + B; }
__device__ __forceinline__ bool may_run_ahead(const Cur& g, const Cur& d, int B) { return item_may_run_ahead(g.item, d.item, B); }
__device__ __forceinline__ void cur_next(Cur& k, const Env& e) {
    ++k.seq;
    if (++k.i < k.run.ntiles) return;
    if (!item_ext(e, k.l)) ++k.use;
    ++k.ni;
    ++k.item;
    cur_seek(k, e);
}

// The order in which every role takes a cluster's tiles: the gate/up part of the first tile, then per tile its down
// part, with the next tile's gate/up part before it when that may run ahead and after it otherwise.  Written as a state
// machine so that each part's code exists once per role (inlined at one call site).
template <class FS, class FG, class FD>
__device__ __forceinline__ void walk_tiles(const Env& env, int B, FS stop, FG gate_up, FD down) {
    Cur g, d;
    cur_init(g, env);
    d = g;
    int st = g.valid ? 3 : 0;                                      // 3: the very first gate/up part; 0: start of a round
    for (;;) {
        bool is_g;
        if (st == 3) { is_g = true; st = 0; }
        else if (st == 0) {
            if (!d.valid || stop()) break;
            if (g.valid && !env.serial && may_run_ahead(g, d, B)) { is_g = true; st = 1; } else { is_g = false; st = 2; }
        } else if (st == 1) { is_g = false; st = 0; }               // the down part behind a gate/up part that ran ahead
        else { st = 0; if (!g.valid) continue; is_g = true; }       // the gate/up part behind the down part
        if (is_g) { gate_up(g); cur_next(g, env); } else { down(d); cur_next(d, env); }
    }
}

// Shared memory: a fixed head (item counts, the tiles' neuron ids, barriers), the exchange area of the GLU, the weight
// ring (six or eight stages, decided at the start of the launch), then the h tile and the x ring, which share what is
// left: the h tile is sized for the largest tile of the step; the x ring takes the rest, or lies over the h tile.
template <int HS8>
struct Geo {
    static constexpr int H = 8 * HS8;
    // weight ring stages: six, or eight when the x ring lies over the h tile (one episode, one tile per layer) and can
    // spare the room.  (Measured at H = 2048, top-20 % / full list, before that mode existed: 4 stages 420 / 1344 us per
    // step, 5: 401 / 1288, 6: 398 / 1264.)  The x ring takes what the weight ring and the h tile leave.
    static constexpr int NW_MIN = 6, NW_MAX = 8;
    static constexpr int NSB = HS8 / 64;               // 64-column boxes per column slice
    static constexpr int NMB = HS8 / 128;              // 128-column output blocks per slice
    static constexpr int NCH = H / 64;                 // 64-column blocks of H
    static constexpr int SPS = SB / (HS8 * 2);         // slots (neurons) of one down stage: 32 or 64
    static constexpr int KPS = SPS / 16;               // product steps of one down stage
    static constexpr int ND2 = NMB == 1 ? 2 : 1;       // down accumulators (an item's flush overlaps the next item's products)
    static constexpr int D2_COL = 4 * NTOK;            // tensor memory: D1[2] at 0 and 128 (128 columns each), D2 from 256
    static constexpr int OFF_K = 0;                    // counts of the items
    static constexpr int OFF_P = OFF_K + MAX_ITEMS * 4;         // (OFF_K: the items' counts, then this cluster's run lengths; OFF_P: run starts)
    static constexpr int OFF_IDX = OFF_P + MAX_ITEMS * 4;       // neuron ids of three tiles in turn
    static constexpr int OFF_REC = OFF_IDX + 3 * CT * 4;
    static constexpr int OFF_MISC = OFF_REC + 4 * NT * 4;
    static constexpr int OFF_BAR = OFF_MISC + 128;
    static constexpr int OFF_EX = 9 * 1024;
    static constexpr int OFF_W = OFF_EX + EXCH;                // weight ring, then the h tile and the x ring up to END
    static constexpr int END = 231424;
    static constexpr int TOTAL = END + 1024;           // + slack for the 1024-byte alignment
    static_assert(OFF_BAR + 640 <= OFF_EX, "fixed head overflows");
    static_assert(TOTAL <= 232448, "buffers exceed the shared memory of a CTA");
};

template <int HS8, bool EQ4>
__global__ void __launch_bounds__(NTHREADS, 1) step_kernel(const __grid_constant__ PArgs a,
                                                          const __grid_constant__ CUtensorMap tmXext) {
    using G = Geo<HS8>;
    constexpr int H = G::H, NSB = G::NSB, NMB = G::NMB, SPS = G::SPS, KPS = G::KPS, ND2 = G::ND2, NCH = G::NCH;
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* gbase = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t sW = base + G::OFF_W;
    int* sK = reinterpret_cast<int*>(gbase + G::OFF_K);
    int* sP = reinterpret_cast<int*>(gbase + G::OFF_P);
    int* sIdx = reinterpret_cast<int*>(gbase + G::OFF_IDX);
    float* sRec = reinterpret_cast<float*>(gbase + G::OFF_REC);
    volatile int* sMisc = reinterpret_cast<volatile int*>(gbase + G::OFF_MISC);
    volatile uint32_t* g_tmem = reinterpret_cast<volatile uint32_t*>(gbase + G::OFF_MISC);      // [0] tensor-memory base
    volatile int* sAbort = sMisc + 1;                              // [1] a wait of this CTA gave up
    volatile int* sHslots = sMisc + 2;                             // [2] slots of the h tile (largest tile, rounded to 16)
    volatile int* sLoaded = sMisc + 3;                             // [3] neurons whose gate/up rows the loaders have started on
    int* sReady = const_cast<int*>(sMisc) + 4;                     // [4] ring stages (in consumption order) whose data has landed
    volatile int* sAlias = sMisc + 5;                              // [5] the x ring lies over the h tile (see below)
    const uint32_t s_tmem = base + G::OFF_MISC;
    const uint32_t bar0 = base + G::OFF_BAR;
    auto w_full = [&](int s) { return bar0 + 8 * s; };              // NW <= 6
    auto w_empty = [&](int s) { return bar0 + 96 + 8 * s; };
    auto x_full = [&](int s) { return bar0 + 192 + 8 * s; };        // up to XS_MAX = 8
    auto x_empty = [&](int s) { return bar0 + 320 + 8 * s; };
    auto d1_full = [&](int s) { return bar0 + 448 + 8 * s; };       // 2
    auto d2_full = [&](int s) { return bar0 + 464 + 8 * s; };       // 2
    auto d2_empty = [&](int s) { return bar0 + 480 + 8 * s; };
    auto x_ready = [&](int s) { return bar0 + 496 + 8 * s; };       // 2
    auto x_free = [&](int s) { return bar0 + 512 + 8 * s; };
    const uint32_t h_free = bar0 + 536, g_all = bar0 + 544;
    auto h_arr = [&](int p) { return bar0 + 552 + 8 * p; };        // CS: piece p of the tile's h has arrived in this CTA
    const uint32_t d_local = bar0 + 616;                           // this CTA's down products of a tile are complete

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int j = (int)cluster_ctarank(), c = (int)cluster_id_x(), NC = (int)cluster_count_x();
    const int T = a.T, L = a.L, B = a.B, I = a.I;
    const int n_ctas = (int)gridDim.x;
    const int n_items = L * B;
    const int anchor_mode = EQ4 ? a.anchor_mode : (int)RM_ANCHOR_NONE;

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
    __syncthreads();
    if (tid == 0) {
        for (int s = 0; s < G::NW_MAX; ++s) { mbar_init(w_full(s), 128); mbar_init(w_empty(s), 1); }
        for (int s = 0; s < XS_MAX; ++s) { mbar_init(x_full(s), 2); mbar_init(x_empty(s), 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(d1_full(s), 1); mbar_init(d2_full(s), 1); mbar_init(d2_empty(s), 256);
            mbar_init(x_ready(s), CS); mbar_init(x_free(s), CS);
        }
        for (int p2 = 0; p2 < CS; ++p2) mbar_init(h_arr(p2), 1);
        mbar_init(h_free, CS); mbar_init(g_all, CS); mbar_init(d_local, 1);
        fence_mbar_init();
        *sAbort = 0;
        *sLoaded = 0;
        *sReady = 0;
        sMisc[8] = 16;                                             // [8] largest tile of the step; [9] most tiles of an item
        sMisc[9] = 0;
    }
    __syncthreads();
    {
        // This cluster's run in every item's list: one thread per item (sK holds the counts; afterwards sP the run starts
        // and sK the run lengths).  One thread doing all of them took ~3 us of every launch.
        Run r{0, 0, 0};
        const bool mine = tid < n_items;
        if (mine) {
            const int l = tid / B, b = tid - l * B;
            int S = 0, P = 0;
            for (int b2 = 0; b2 < B; ++b2) {
                const int K2 = sK[l * B + b2];
                S += K2;
                if (b2 < b) P += K2;
            }
            r = cluster_run(sK[tid], P, S, c, NC);
            if (r.ntiles > 0) atomicMax(const_cast<int*>(sMisc) + 8, (r.n + r.ntiles - 1) / r.ntiles);
            atomicMax(const_cast<int*>(sMisc) + 9, r.ntiles);
        }
        __syncthreads();
        if (mine) { sP[tid] = r.start; sK[tid] = r.n; }
        __syncthreads();
    }
    if (tid == 0) {
        *sHslots = (sMisc[8] + 15) & ~15;
        // One episode and the tiles taken strictly one after the other (gate/up, GLU, down): a tile's h is written after
        // its gate/up products and dead before the next tile's x copies start (they wait for this CTA's down products), so
        // the x ring lies over the h tile, and the room that saves goes to the weight ring.  With one tile per layer and
        // cluster nothing is lost by that order.  With several it gives up running the next tile's gate/up products under
        // this tile's GLU and down products: at H = 2048 the deeper rings are worth more (full lists: 1177 -> 1076 us per
        // step), at H = 1024, where a tile's gate/up part is half as long, less (292 -> 320).
        *sAlias = B == 1 && (sMisc[9] <= 1 || HS8 == 256);
    }
    if (warp == W_MMA) tmem_alloc(s_tmem, 512);
    // the x copies bring token rows 0..T-1 only: the other rows of every ring stage stay zero from here on (when the ring
    // lies over the h tile they hold old h values instead: the sums of the token columns T..63 are never used, the
    // epilogue writes zeros for them)
    for (int e = tid; e < (G::END - G::OFF_W - G::NW_MIN * SB) / 16; e += NTHREADS)
        reinterpret_cast<uint4*>(gbase + G::OFF_W + G::NW_MIN * SB)[e] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    // (the cluster's x copies in global memory need no clearing: a copy brings token rows 0..T-1 only)
    tc_fence_before();
    __syncthreads();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem = *g_tmem;
    // r starts as a copy of r_in: cluster 0's CTA j copies column slice j of every episode and counts itself on the
    // episode's copy counter; nobody adds into r before the 8 copies are counted
    const int pre = a.r_in != a.r ? CS : 0;
    if (pre && c == 0 && warp < 8) {
        for (int b = 0; b < B; ++b) {
            const float4* src = reinterpret_cast<const float4*>(a.r_in + (size_t)b * T * H + j * HS8);
            float4* dst = reinterpret_cast<float4*>(a.r + (size_t)b * T * H + j * HS8);
            for (int e = tid; e < T * (HS8 / 4); e += 256) {
                const int t = e / (HS8 / 4), q = e - t * (HS8 / 4);
                dst[(size_t)t * (H / 4) + q] = src[(size_t)t * (H / 4) + q];
            }
            __threadfence();
            named_barrier(1, 256);
            if (tid == 0) red_release_gpu(a.sync + SYNC_COPY + b, 1);
        }
    }
    const int h_half = *sHslots * 128;                             // bytes of the hi block (= of the lo block) of the h tile
    const bool alias = *sAlias != 0;
    const bool alias_multi = alias && sMisc[9] > 1;             // ... and some item has several tiles (see d_local)
    const int NW = alias ? G::NW_MAX : G::NW_MIN;       // (nine with three x stages: 2-5 % slower than eight with four)
    const int OFF_HX = G::OFF_W + NW * SB;
    const uint32_t sH = base + OFF_HX;
    const uint32_t sX = alias ? sH : sH + 2 * h_half;
    int xs_n = (G::END - OFF_HX - (alias ? 0 : 2 * h_half)) / XSB;
    const int XS = xs_n > XS_MAX ? XS_MAX : xs_n;                    // >= 2
    Env env{sP, sK, L, B, c, NC, a.x_ext, alias ? 1 : 0};

    // The kernel is large (every role is its own code) and the instruction caches are small: a wait's slow path and the
    // error report live in functions of their own, and every role calls its per-tile code from one place, so that the
    // loops that run all the time stay compact.
    bool gave_up = false;
    auto timed_out = [&](int line) {
        report_timeout(a.status, sAbort, a.sync, line);
        gave_up = true;
    };
    auto wait_at = [&](uint32_t bar, uint32_t parity, int line) {
        if (gave_up) return;
        if (mbar_test_wait(bar, parity)) return;
        gave_up = wait_slow(bar, parity, line, sAbort, a.sync, a.status);
    };
#define WAIT(bar, parity) wait_at((bar), (parity), __LINE__)

    const uint64_t desc_k = smem_desc_sw128(0, 16, 1024);
    const uint64_t desc_mn_a = smem_desc_sw128(0, SPS * 128, 1024);
    const uint64_t desc_mn_b = smem_desc_sw128(0, (uint32_t)h_half, 1024);
    constexpr uint32_t IDESC_G = idesc_bf16_f32(128, 2 * NTOK, false, false);
    constexpr uint32_t IDESC_D = idesc_bf16_f32(128, 2 * NTOK, true, true);

    if (warp >= W_LOAD0 && warp < W_LOAD0 + 4) {
        // ================================================================ loaders: the step's weight rows, in the
        // order in which the issuer consumes them
        const int lt = tid - W_LOAD0 * 32, lw = lt >> 5;
        const int pc = lt & 7, r0 = lt >> 3;                       // gate/up: 16-byte piece, rows r0 + 16 q
        int ws = 0;                                                // ring slot of the next stage; its pass over the ring
        uint32_t wpass = 0;
        auto advance = [&]() { if (++ws == NW) { ws = 0; ++wpass; } };
        int loaded = 0;
        bool stop = false;                                         // agreed by all loader threads at the start of a tile
        // one lane per warp waits for the stage (128 threads testing one mbarrier take several hundred clocks)
        auto acquire = [&]() {
            if (wpass >= 1) {
                if (lane == 0) WAIT(w_empty(ws), (wpass - 1) & 1);
                __syncwarp();
            }
            return sW + ws * SB;
        };
        auto load_g = [&](const Cur& k) {
            int t0, ts, off, nj;
            tile_span(k.run, k.i, t0, ts);
            cta_span(ts, j, off, nj);
            // the tile's neuron ids, for these rows and for the tile's down stages
            const int32_t* list = a.idx ? a.idx + (size_t)k.b * a.idx_b_stride + (size_t)k.l * a.idx_l_stride : nullptr;
            int* ids = sIdx + (k.seq % 3) * CT;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int kk = lt + 128 * e;
                int n = -1;
                if (kk < ts) {
                    n = list ? __ldg(list + t0 + kk) : t0 + kk;
                    if (n < 0 || n >= I) { rm_set_status(a.status, RM_ERR_INDEX); n = -1; }
                }
                ids[kk] = n;
            }
            stop = named_barrier_or(3, 128, gave_up || *sAbort);
            if (lt == 0) { loaded += nj; *sLoaded = loaded; }
            const __nv_bfloat16* src[4];
            bool ok[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = r0 + 16 * q, i = r >> 1;
                const int n = i < nj ? ids[off + i] : -1;
                ok[q] = n >= 0;
                src[q] = a.packed[k.l] + (size_t)(n < 0 ? 0 : n) * 3 * H + (r & 1) * HS8 + pc * 8;
            }
            // stage cc: the rows over the 64-column blocks cc (first 8 KB) and cc + NCH/2 (second 8 KB)
            for (int cc = 0; cc < NCH / 2; ++cc) {
                const uint32_t st = acquire();
                if (lt == 0) RM_TR(k.item, 0, cc);
                const int c1 = cc + NCH / 2;
                const int so0 = (cc / NSB) * 3 * HS8 + (cc % NSB) * 64, so1 = (c1 / NSB) * 3 * HS8 + (c1 % NSB) * 64;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int r = r0 + 16 * q;
                    const uint32_t d = st + (r >> 3) * 1024 + (r & 7) * 128 + ((pc ^ (r & 7)) << 4);
                    if (ok[q]) {
                        cp_async16(d, src[q] + so0, true);
                        cp_async16(d + 8192, src[q] + so1, true);
                    }
                }
                if (lt == 0) RM_TR(k.item, 1, cc);
                cp_async_arrive_noinc(w_full(ws));
                advance();
            }
        };
        auto load_d = [&](const Cur& k) {
            int t0, ts;
            tile_span(k.run, k.i, t0, ts);
            const int* ids = sIdx + (k.seq % 3) * CT;
            const int kst = (ts + 15) >> 4, nst = (ts + SPS - 1) / SPS;
            constexpr int PPS = HS8 / 8;                           // 16-byte pieces of a neuron's down slice
            constexpr int SPW = 32 / PPS;                          // slots one warp instruction covers
            const int piece = lane % PPS;
            const __nv_bfloat16* wl = a.packed[k.l] + j * 3 * HS8 + 2 * HS8 + piece * 8;
            const int s0 = d_stage_first(ts, j, SPS, nst);
            for (int ks0 = 0; ks0 < nst; ++ks0) {
                const int s = d_stage(s0, ks0, nst);
                const uint32_t st = acquire();
#pragma unroll
                for (int m = 0; m < 8; ++m) {
                    const int slot = (lw + 4 * m) * SPW + lane / PPS, kk = SPS * s + slot;
                    if (kk >= 16 * kst) continue;                  // beyond the last product step of the tile
                    const int n = kk < ts ? ids[kk] : -1;
                    const uint32_t d = st + (piece >> 3) * (SPS * 128) + slot * 128 + (((piece & 7) ^ (slot & 7)) << 4);
                    cp_async16(d, wl + (size_t)(n < 0 ? 0 : n) * 3 * H, n >= 0);      // unused slots of the last step: zeros
                }
                cp_async_arrive_noinc(w_full(ws));
                advance();
            }
        };
        walk_tiles(env, B, [&]() { return stop; }, load_g, load_d);
        cp_async_wait<0>();
    } else if (warp == W_PF) {
        // ================================================================ L2 prefetch: while the loaders wait for ring
        // space (the arithmetic is held up at a layer boundary), the rows of the tiles ahead are asked into L2, so
        // that HBM keeps streaming.  A CTA asks for the whole rows of its own neurons; the cluster's CTAs together
        // cover every slice that any of them will read.
        Cur k;
        cur_init(k, env);
        int asked = 0;
        const int ahead_n = a.pf_bytes / (6 * H);
        while (k.valid && a.pf_bytes > 0) {
            int t0, ts, off, nj;
            tile_span(k.run, k.i, t0, ts);
            cta_span(ts, j, off, nj);
            bool go = false;
            for (uint32_t i = 0; i < (1u << 20); ++i) {
                if (asked - *sLoaded <= ahead_n) { go = true; break; }
                if (*sAbort) break;
                __nanosleep(200);
            }
            if (!go) break;                                        // a hint only: giving up costs nothing
            if (lane < nj) {
                const int32_t* list = a.idx ? a.idx + (size_t)k.b * a.idx_b_stride + (size_t)k.l * a.idx_l_stride : nullptr;
                const int n = list ? __ldg(list + t0 + off + lane) : t0 + off + lane;
                if (n >= 0 && n < I) prefetch_l2(a.packed[k.l] + (size_t)n * 3 * H, 6 * H);
            }
            asked += nj;
            cur_next(k, env);
        }
    } else if (warp >= W_X0 && warp < W_X0 + NXW) {
        // ================================================================ x copies: one thread of each of four warps,
        // block n of the stream by thread n mod 4.  The cluster's own x is stored as shared-memory images, so a block
        // is one contiguous 8 KB copy; the caller's x (single-layer entry) comes as one tensor-map box.
        if (lane == 0) {
            // thread xq copies the half (xq & 1) of every second stage, starting with stage xq >> 1
            const int xq = warp - W_X0, half = xq & 1;
            uint32_t n = xq >> 1, ph = 0;                          // stage number in the stream; ring pass parity
            int xs = (xq >> 1) % XS;                               // (XS >= 2)
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
                        const uint32_t rph = (k.use >> 1) & 1;
                        bool ok = false;
                        for (uint32_t i = 0; i < (1u << 22) && !ok; ++i) {
                            ok = mbar_try_wait_cluster(x_ready(slot), rph);
                            if (!ok && i > 64) __nanosleep(32);
                            if ((i & 1023u) == 1023u && *sAbort) break;
                        }
                        if (!ok) { if (!*sAbort) timed_out(__LINE__); gave_up = true; break; }
                        if (xq == 0) RM_PS(k.item, 0);
                    }
                }
                const unsigned char* img = reinterpret_cast<const unsigned char*>(a.xbuf) + (size_t)(c * 2 + slot) * NCH * X_BYTES;
                // (x ring over the h tile: the previous tile's h is read until this CTA's down products are complete.  With one
                // tile per layer the next tile's x exists only after every CTA's adds of this layer, so nothing to wait for.)
                if (alias_multi && k.seq >= 1) WAIT(d_local, (k.seq - 1) & 1);
                for (int cc = xq >> 1; cc < NCH / 2; cc += 2) {
                    if (n >= (uint32_t)XS) WAIT(x_empty(xs), ph ^ 1);
                    if (half == 0) RM_TR(k.item, 2, cc);
                    const int blk = cc + half * (NCH / 2);
                    const uint32_t dst = sX + xs * XSB + half * X_BYTES;
                    if (ext) {
                        mbar_arrive_expect_tx(x_full(xs), X_BYTES);
                        tma_load_2d(dst, &tmXext, blk * 64, 0, x_full(xs));
                    } else {
                        mbar_arrive_expect_tx(x_full(xs), (uint32_t)T * 128u);
                        bulk_load(dst, img + (size_t)blk * X_BYTES, (uint32_t)T * 128u, x_full(xs));
                    }
                    n += 2;
                    xs += 2;
                    if (xs >= XS) { xs -= XS; ph ^= 1; }
                }
                cur_next(k, env);
            }
        }
    } else if (warp == W_WATCH) {
        // ================================================================ stage watcher (one thread): waits for the ring
        // stages in the order in which the issuer consumes them, fences their cp.async data for the tensor core, and
        // publishes the count
        if (lane == 0) {
            uint32_t wph = 0, xph = 0, stage = 0;                  // parities of the ring passes; stages published
            int ws = 0;
            int xs = 0;
            auto watch_g = [&](const Cur& k) {
                long long c_w = 0, c_x = 0, c_f = 0;
                for (int cc = 0; cc < NCH / 2; ++cc) {
                    const long long q0 = RM_CLK();
                    const uint32_t both = mbar_test_wait_2(w_full(ws), wph, x_full(xs), xph);
                    if (!(both & 1u)) WAIT(w_full(ws), wph);
                    const long long q1 = RM_CLK();
                    RM_TR(k.item, 3, cc);
                    if (!(both & 2u)) WAIT(x_full(xs), xph);
                    const long long q2 = RM_CLK();
                    RM_TR(k.item, 4, cc);
                    fence_proxy_async_smem();
                    st_release_cta(sReady, (int)++stage);
                    const long long q3 = RM_CLK();
                    if (cc > 0) { c_w += q1 - q0; c_x += q2 - q1; c_f += q3 - q2; }
                    if (++xs == XS) { xs = 0; xph ^= 1; }
                    if (++ws == NW) { ws = 0; wph ^= 1; }
                }
                if (k.i == 0) { RM_PC(k.item, 13, c_w); RM_PC(k.item, 14, c_x); RM_PC(k.item, 15, c_f); }
            };
            auto watch_d = [&](const Cur& k) {
                int t0, ts;
                tile_span(k.run, k.i, t0, ts);
                const int nst = (ts + SPS - 1) / SPS;
                const int s0 = d_stage_first(ts, j, SPS, nst);
                uint32_t arrived = 0;                              // pieces of this tile's h known to be here
                for (int ks0 = 0; ks0 < nst; ++ks0) {
                    const uint32_t want = d_stage_pieces(ts, d_stage(s0, ks0, nst), SPS);
                    bool w_ok;
                    if (want & ~arrived) {
                        // the stage's weights and all eight pieces in one round of tests
                        const uint32_t m = mbar_test_wait_8_1(h_arr(0), k.seq & 1, w_full(ws), wph);
                        arrived |= m & 0xffu;
                        w_ok = (m >> 8) & 1u;
                    } else {
                        w_ok = mbar_test_wait(w_full(ws), wph);
                    }
                    if (!w_ok) WAIT(w_full(ws), wph);
                    for (uint32_t i = 0; (want & ~arrived) && i < (1u << 20) && !gave_up; ++i) {
                        arrived |= mbar_test_wait_8_1(h_arr(0), k.seq & 1, w_full(ws), wph) & 0xffu;
                        if ((i & 255u) == 255u && *sAbort) gave_up = true;
                    }
                    if ((want & ~arrived) && !gave_up) timed_out(__LINE__);
                    fence_proxy_async_smem();
                    st_release_cta(sReady, (int)++stage);
                    RM_TR(k.item, 11, ks0);
                    if (++ws == NW) { ws = 0; wph ^= 1; }
                }
            };
            walk_tiles(env, B, [&]() { return gave_up; }, watch_g, watch_d);
        }
    } else if (warp == W_MMA) {
        // ================================================================ issuer (one warp; an elected lane issues)
        // Issuing is the scarce resource here: the tensor pipe idles while the issuing thread executes anything else
        // (4 products of a stage keep it busy for ~256 clocks; a commit adds ~30-50, an acquire load ~160, a test of an
        // mbarrier ~170, and in a loop that only lane 0 of a warp runs every branch around a wait loop cost another
        // ~100-170 per stage).  Hence: the whole warp runs the control flow and one elected lane issues (measured 100-150
        // clocks per stage cheaper than a one-lane loop); the watcher thread does the waiting and the proxy fence and
        // publishes how many stages of the stream have landed; the issuer reads that count with a relaxed load (in a
        // function of its own, off the hot path) only when it has used up what it knows of.
        {
            int ws = 0, xs = 0;                                    // ring slots of the next weight stage and x stage
            const uint64_t dW0 = desc_k | desc_addr(sW), dX0 = desc_k | desc_addr(sX), dA0 = desc_mn_a | desc_addr(sW);
            uint32_t stage = 0, ready = 0;                         // stages issued; stages known to have landed
            auto need = [&](int line) {
                if (stage < ready || gave_up) return;
                ready = (uint32_t)ld_relaxed_cta(sReady);            // (a call costs ~200 clocks here: look once before it)
                if (stage < ready) return;
                ready = landed_stages(sReady, stage, const_cast<const int*>(sAbort));
                if (stage < ready) return;
                if (*sAbort) { gave_up = true; return; }
                if (lane == 0) timed_out(line);
                gave_up = true;
            };
            auto issue_g = [&](const Cur& k) {
                const uint32_t d1 = tmem + (k.seq & 1) * (2 * NTOK);
                for (int cc = 0; cc < NCH / 2; ++cc) {
                    if (lane == 0) RM_TR(k.item, 7, cc);
                    need(__LINE__);
                    if (lane == 0) RM_TR(k.item, 8, cc);
                    if (cc == 0 && k.i == 0 && lane == 0) RM_PS(k.item, 1);
                    tc_fence_after();
                    if (lane == 0) RM_TR(k.item, 9, cc);
                    const uint64_t da = dW0 + (uint64_t)(ws * (SB >> 4)), db = dX0 + (uint64_t)(xs * (XSB >> 4));
                    if (elect_one()) {
                        RM_TR(k.item, 5, cc);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) mma_bf16_ss(d1, da + 2 * ks, db + 2 * ks, IDESC_G, (cc | ks) != 0);
                        mma_commit(x_empty(xs));
                        mma_commit(w_empty(ws));
                        RM_TR(k.item, 6, cc);
                    }
                    __syncwarp();
                    if (lane == 0) RM_TR(k.item, 10, cc);
                    if (++xs == XS) xs = 0;
                    if (++ws == NW) ws = 0;
                    ++stage;
                }
                if (elect_one()) {
                    mma_commit(d1_full(k.seq & 1));
                    if (alias) mma_commit_mc(g_all, 0xff);            // this CTA's x ring (which lies over its h tile) is read out
                    if (k.i == 0) RM_PS(k.item, 24);
                    if (k.i == k.run.ntiles - 1 && !item_ext(env, k.l)) mma_commit_mc(x_free(k.use & 1), 0xff);
                }
                __syncwarp();
            };
            auto issue_d = [&](const Cur& k) {
                int t0, ts;
                tile_span(k.run, k.i, t0, ts);
                const int kst = (ts + 15) >> 4, nst = (ts + SPS - 1) / SPS;
                const int d2b = ND2 == 2 ? (k.ni & 1) : 0, nu = ND2 == 2 ? (k.ni >> 1) : k.ni;
                if (k.i == 0 && nu >= 1) WAIT(d2_empty(d2b), (nu - 1) & 1);
                const uint32_t d2 = tmem + G::D2_COL + d2b * (2 * NTOK);
                const uint64_t dh0 = desc_mn_b | desc_addr(sH);      // 16 slots of h per product step
                // (the watcher publishes a down stage only when the h pieces it reads have arrived; the stages come in
                // the order of d_stage)
                const int s0 = d_stage_first(ts, j, SPS, nst);
                for (int ks0 = 0; ks0 < nst; ++ks0) {
                    const int s = d_stage(s0, ks0, nst);
                    if (lane == 0) RM_TR(k.item, 14, ks0);
                    need(__LINE__);
                    if (ks0 == 0 && lane == 0) RM_PS(k.item, 4);
                    tc_fence_after();
                    if (lane == 0) RM_TR(k.item, 12, ks0);
                    const uint64_t da = dA0 + (uint64_t)(ws * (SB >> 4)), dh = dh0 + (uint64_t)(s * (KPS * (2048 >> 4)));
                    if (elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < KPS; ++ks) {
                            if (KPS * s + ks < kst) {
#pragma unroll
                                for (int mb = 0; mb < NMB; ++mb)
                                    mma_bf16_ss(d2 + mb * (2 * NTOK), da + (uint64_t)((mb * (2 * SPS * 128) + ks * 2048) >> 4),
                                                dh + (uint64_t)(ks * (2048 >> 4)), IDESC_D, !(k.i == 0 && ks0 == 0 && ks == 0));
                            }
                        }
                        mma_commit(w_empty(ws));
                    }
                    __syncwarp();
                    if (lane == 0) RM_TR(k.item, 13, ks0);
                    if (++ws == NW) ws = 0;
                    ++stage;
                }
                if (elect_one()) {
                    if (alias_multi) mma_commit(d_local);
                    mma_commit_mc(h_free, 0xff);
                    if (k.i == k.run.ntiles - 1) { mma_commit(d2_full(d2b)); RM_PS(k.item, 25); }
                }
                __syncwarp();
            };
            walk_tiles(env, B, [&]() { return gave_up; }, issue_g, issue_d);
        }
    } else {
        // ================================================================ epilogue (8 warps): GLU, h exchange, flush
        const int et = tid;                                         // 0..255
        const int q4 = warp & 3, ch = warp >> 2;                    // tensor-memory lane quarter; token half
        // D1 (M = 128): lane m < 64 holds row m's sum over the first half of H (token columns 0..63), lane 64 + m the
        // same row's sum over the second half (token columns 64..127).  Row 2 i is neuron i's gate, row 2 i + 1 its up.
        const bool fin = q4 < 2;                                    // lanes with a first-half sum (the others: second half)
        const int m_row = (q4 & 1) * 32 + lane;                     // row 0..63 of this lane
        const int ni_loc = m_row >> 1;                              // neuron of this lane among the CTA's 32
        const bool isup = lane & 1;
        float* sEx = reinterpret_cast<float*>(gbase + G::OFF_EX);   // [direction][token half][16 tokens][64 rows] fp32
        unsigned char* gH = gbase + OFF_HX;
        int seq = 0, ni = 0;
        bool stop = false;
        // Normalisation of an item's input into this cluster's copy of x: CTA j takes the token rows j, j + 8, ...,
        // one row per warp.  With one episode it runs right before the item's tiles (it has to wait for the previous
        // layer's adds anyway); with several episodes it runs one item ahead, so that the next item's gate/up
        // products can start while this item's tiles are finished.
        int use = 0;
        auto norm_item = [&](int item) {
            const int l = item / B, b = item - l * B;
            const int slot = use & 1, nu = use >> 1;
            ++use;
            const bool xf_ok = nu >= 1 ? mbar_test_wait(x_free(slot), (nu - 1) & 1) : true;     // looked at before the stores
            if (l > 0) {
                // every CTA has added its part of layer l-1 to this episode's rows
                const int target = a.per_item ? n_ctas : a.sync_base[b] + n_ctas * l;
                const int* counter = a.per_item ? a.sync + SYNC_ITEM + (l - 1) * B + b : a.sync + b;
                // one thread per CTA watches the counter (with every warp's lane 0 polling, ~1000 threads read the line
                // that the last arrivals have to get through); the barrier passes its acquire on to the others
                if (et == 0 && !gave_up) {
                    bool ok = false;
                    for (uint32_t i = 0; i < (1u << 21); ++i) {
                        if (ld_acquire_gpu(counter) >= target) { ok = true; break; }
                        if ((i & 255u) == 255u && (*sAbort || ld_acquire_gpu(a.sync + SYNC_ABORT))) break;
                    }
                    if (!ok) { if (!*sAbort && !ld_acquire_gpu(a.sync + SYNC_ABORT)) timed_out(__LINE__); gave_up = true; *sAbort = 1; }
                }
                named_barrier(1, 256);
            }
            if (et == 0) RM_PS(item, 8);
            const long long n0 = RM_CLK();
            long long n1 = n0, n2 = n0, n3 = n0;
            const int row = j + 8 * warp;
            if (row < T) {
                const float4* src = reinterpret_cast<const float4*>((l == 0 ? a.r_in : a.r) + ((size_t)b * T + row) * H);
                float4 v[H / 128];
                float ss = 0.f;
#pragma unroll
                for (int q = 0; q < H / 128; ++q) v[q] = __ldcg(src + lane + 32 * q);
#pragma unroll
                for (int q = 0; q < H / 128; ++q) {
                    ss = fmaf(v[q].x, v[q].x, ss); ss = fmaf(v[q].y, v[q].y, ss);
                    ss = fmaf(v[q].z, v[q].z, ss); ss = fmaf(v[q].w, v[q].w, ss);
                }
#pragma unroll
                for (int dd = 16; dd > 0; dd >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, dd);
                const float inv = 1.0f / sqrtf(ss / (float)H + 1e-6f);
                n1 = RM_CLK();
                if (!xf_ok) WAIT(x_free(slot), (nu - 1) & 1);          // the products that read this copy's previous contents are complete
                // columns 4 (lane + 32 q) .. + 3 of this row: block q * 2 + lane / 16, 16-byte piece (lane % 16) / 2 of the
                // row's 128 bytes in that block, swizzled by the row
                unsigned char* img = reinterpret_cast<unsigned char*>(a.xbuf) + (size_t)(c * 2 + slot) * (H / 64) * X_BYTES +
                                     row * 128 + ((((lane & 15) >> 1) ^ (row & 7)) << 4) + (lane & 1) * 8;
#pragma unroll
                for (int q = 0; q < H / 128; ++q) {
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(v[q].x * inv, v[q].y * inv);
                    const __nv_bfloat162 hi = __floats2bfloat162_rn(v[q].z * inv, v[q].w * inv);
                    uint2 u;
                    u.x = *reinterpret_cast<const uint32_t*>(&lo);
                    u.y = *reinterpret_cast<const uint32_t*>(&hi);
                    *reinterpret_cast<uint2*>(img + (size_t)(2 * q + (lane >> 4)) * X_BYTES) = u;
                }
                n2 = RM_CLK();
                // the readers are copy-engine reads issued by this cluster's CTAs after the cluster-scope arrivals below
                fence_proxy_async_global();
                n3 = RM_CLK();
            }
            stop = named_barrier_or(1, 256, gave_up || *sAbort);
            const long long n4 = RM_CLK();
            if (warp == 0 && lane < CS) mbar_arrive_remote(map_to_rank(x_ready(slot), lane));
            // This CTA's reads of the item's input rows are complete (their values went into the sums above).  The adds
            // of the item's OWN results go into the same rows, and a faster cluster's adds wait for this count.
            if (et == 32) red_release_gpu(a.per_item ? a.sync + SYNC_RITEM + item : a.sync + SYNC_READ + b, 1);
            if (et == 0) { RM_PS(item, 9); RM_PC(item, 26, n1 - n0); RM_PC(item, 27, n2 - n1); RM_PC(item, 28, n3 - n2); RM_PC(item, 29, n4 - n3); RM_PC(item, 30, RM_CLK() - n4); }
        };
        // x of a non-empty item is prepared right before the item's own tiles, or one non-empty item earlier when the
        // issuer may run that item's gate/up products ahead (item_may_run_ahead)
        int normed = -1;                                            // last item whose x has been prepared
        for (int item = 0; item < n_items && !stop; ++item) {
            if (item_run(env, item).ntiles > 0) {
                // (one call site for the normalisation: first this item, then the look-ahead item if there is one)
                int q = item;
                for (int pass = 0; pass < 2 && !stop; ++pass) {
                    if (pass == 1) {
                        q = item + 1;
                        while (q < n_items && q < item + B && item_run(env, q).ntiles == 0) ++q;
                        if (!(q < n_items && q < item + B)) break;
                    }
                    if (q > normed) {
                        normed = q;
                        if (!item_ext(env, q / B)) norm_item(q);
                    }
                }
            }
            if (stop) break;
            const int l = item / B, b = item - l * B;
            const Run run = item_run(env, item);
            const int32_t* list = a.idx ? a.idx + (size_t)b * a.idx_b_stride + (size_t)l * a.idx_l_stride : nullptr;
            for (int i = 0; i < run.ntiles && !stop; ++i, ++seq) {
                int t0, ts, off, nj;
                tile_span(run, i, t0, ts);
                cta_span(ts, j, off, nj);
                const int buf = seq & 1;
                int n = -1;
                if (ni_loc < nj) {
                    n = list ? __ldg(list + t0 + off + ni_loc) : t0 + off + ni_loc;
                    if (n < 0 || n >= I) n = -1;
                }
                const int tok0 = 8 * (ch * 4 + (fin ? 0 : 2) + (isup ? 1 : 0));     // first of this lane's 8 tokens (see below)
                // update steps: the neuron's anchor values for this lane's tokens, asked for before the products are waited for
                float4 ha0 = make_float4(0.f, 0.f, 0.f, 0.f), ha1 = ha0;
                float* hap = nullptr;
                if (EQ4 && anchor_mode != RM_ANCHOR_NONE && n >= 0) {
                    hap = a.h_anchor + (((size_t)l * B + b) * I + n) * a.h_stride + tok0;
                    if (anchor_mode == RM_ANCHOR_UPDATE) {
                        if (tok0 < T) ha0 = __ldcg(reinterpret_cast<const float4*>(hap));
                        if (tok0 + 4 < T) ha1 = __ldcg(reinterpret_cast<const float4*>(hap) + 1);
                    }
                }
                WAIT(d1_full(buf), (seq >> 1) & 1);
                tc_fence_after();
                if (et == 0 && i == 0) RM_PS(item, 2);
                const long long e0 = RM_CLK();
                // the test of "every CTA is done with the previous tile's h" takes ~300 clocks to come back even when the
                // phase is long complete: start it now, look at the result when the h values are ready to be written
                const bool hf_ok = seq >= 1 ? mbar_test_wait(h_free, (seq - 1) & 1) : true;
                float v[32];
                tmem_ld32(tmem + buf * (2 * NTOK) + (fin ? 0 : NTOK) + ch * 32 + ((uint32_t)(q4 * 32) << 16), v);
                tc_fence_before();
                // This lane holds one half's sum of row m_row for tokens 32 ch .. 32 ch + 31.  Of these the first-half
                // lane finishes tokens 0..15 and the second-half lane tokens 16..31: each passes the other 16 values.
                {
                    float* out = sEx + (((fin ? 0 : 1) * 2 + ch) * 16) * 64 + m_row;
#pragma unroll
                    for (int r = 0; r < 16; ++r) out[r * 64] = fin ? v[16 + r] : v[r];
                }
                const long long e1 = RM_CLK();
                named_barrier(1, 256);
                const long long e2 = RM_CLK();
                float s16[16];
                {
                    const float* in = sEx + (((fin ? 1 : 0) * 2 + ch) * 16) * 64 + m_row;
#pragma unroll
                    for (int r = 0; r < 16; ++r) s16[r] = (fin ? v[r] : v[16 + r]) + in[r * 64];
                }
                // lane pair (2 i, 2 i + 1) = (gate row, up row) of neuron i for these 16 tokens: the even lane finishes
                // the first 8 of them, the odd lane the last 8
                float hv[8];
                {
                    float gg[8], uu[8], e[8];
#pragma unroll
                    for (int r = 0; r < 8; ++r) {
                        const float mine = isup ? s16[r] : s16[8 + r];
                        const float got = __shfl_xor_sync(0xffffffffu, mine, 1);
                        gg[r] = isup ? got : s16[r];
                        uu[r] = isup ? s16[8 + r] : got;
                    }
#pragma unroll
                    for (int r = 0; r < 8; ++r) e[r] = __expf(-1.5957691216057308f * (gg[r] + 0.044715f * gg[r] * gg[r] * gg[r]));
#pragma unroll
                    for (int r = 0; r < 8; ++r) e[r] = __fdividef(gg[r], 1.0f + e[r]);
#pragma unroll
                    for (int r = 0; r < 8; ++r) hv[r] = n >= 0 && tok0 + r < T ? e[r] * uu[r] : 0.f;
                }
                if (a.record) {
                    float rec = 0.f;
#pragma unroll
                    for (int r = 0; r < 8; ++r) rec += fabsf(hv[r]);
                    rec += __shfl_xor_sync(0xffffffffu, rec, 1);
                    const int grp = ch * 2 + (fin ? 0 : 1);                  // the four token quarters of a neuron
                    if (grp != 0 && !isup) sRec[grp * NT + ni_loc] = rec;
                    named_barrier(1, 256);
                    if (grp == 0 && !isup && n >= 0) {
                        rec += sRec[NT + ni_loc] + sRec[2 * NT + ni_loc] + sRec[3 * NT + ni_loc];
                        const float sc = a.record_scale ? a.record_scale[(size_t)l * I + n] : 1.f;
                        a.record[(size_t)b * a.rec_b_stride + (size_t)l * I + n] = a.record_scale ? rec * sc : rec;
                    }
                }
                if (EQ4 && hap) {
                    // Eq. 4: the anchor step retains h (fp32, before the split); an update step multiplies the down rows
                    // with h - h_a.  (The record above is that of h itself.)
                    if (anchor_mode == RM_ANCHOR_WRITE) {
                        if (tok0 < T) *reinterpret_cast<float4*>(hap) = make_float4(hv[0], hv[1], hv[2], hv[3]);
                        if (tok0 + 4 < T) *(reinterpret_cast<float4*>(hap) + 1) = make_float4(hv[4], hv[5], hv[6], hv[7]);
                    } else {
                        const float hs[8] = {ha0.x, ha0.y, ha0.z, ha0.w, ha1.x, ha1.y, ha1.z, ha1.w};
#pragma unroll
                        for (int r = 0; r < 8; ++r)
                            if (tok0 + r < T) hv[r] -= hs[r];
                    }
                }
                const long long e3 = RM_CLK();
                if (!hf_ok) WAIT(h_free, (seq - 1) & 1);             // every CTA's down products of the previous tile are complete
                const long long e4 = RM_CLK();
                // The piece barriers complete once per tile: a peer's piece by its two copies (hi and lo rows), armed here
                // (the previous tile's pieces have all arrived: its down products are complete); this CTA's own piece
                // and empty pieces by an arrival alone (the own one further down, behind the writes).
                if (et < CS && et != j) {
                    int poff, pn;
                    cta_span(ts, et, poff, pn);
                    if (pn == 0) mbar_arrive(h_arr(et));
                    else mbar_arrive_expect_tx(h_arr(et), (uint32_t)pn * 256u);
                }
                // (x ring over the h tile: a peer's h tile is free only once its own gate/up products are complete; the
                // test is started here and looked at when the copies are ready to go)
                const bool ga_ok = alias && et < 2 * (CS - 1) ? mbar_test_wait(g_all, seq & 1) : true;
                if (ni_loc < nj) {
                    const int kslot = off + ni_loc;
                    const int p0 = ch * 4 + (fin ? 0 : 2) + (isup ? 1 : 0);   // 16-byte piece (8 tokens) of the row's 128 bytes
                    uint32_t hi[4], lo[4];
#pragma unroll
                    for (int e2i = 0; e2i < 4; ++e2i) {
                        const float f0 = hv[2 * e2i], f1 = hv[2 * e2i + 1];
                        const __nv_bfloat162 h2 = __floats2bfloat162_rn(f0, f1);
                        const float2 hf = __bfloat1622float2(h2);
                        const __nv_bfloat162 l2 = __floats2bfloat162_rn(f0 - hf.x, f1 - hf.y);
                        hi[e2i] = *reinterpret_cast<const uint32_t*>(&h2);
                        lo[e2i] = *reinterpret_cast<const uint32_t*>(&l2);
                    }
                    unsigned char* rowp = gH + kslot * 128 + ((p0 ^ (kslot & 7)) << 4);
                    *reinterpret_cast<uint4*>(rowp) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<uint4*>(rowp + h_half) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                }
                {
                    // slots from ts to the end of the last product step: zeros (their weight rows are zeros too)
                    const int prow = ts + (et >> 4), pp = et & 15;
                    if (prow < (((ts + 15) >> 4) << 4))
                        *reinterpret_cast<uint4*>(gH + (pp >> 3) * h_half + prow * 128 + ((pp & 7) << 4)) = make_uint4(0u, 0u, 0u, 0u);
                }
                const long long e5 = RM_CLK();
                fence_proxy_async_smem();
                const long long e6 = RM_CLK();
                stop = named_barrier_or(1, 256, gave_up || *sAbort);
                const long long e7 = RM_CLK();
                if (et == 0) mbar_arrive(h_arr(j));                  // this CTA's own piece: written, fenced, behind the barrier
                if (et < 2 * (CS - 1) && nj > 0) {
                    if (!ga_ok) WAIT(g_all, seq & 1);
                    // CTA j sends to j + 1, j + 2, ... in turn: the copies of a CTA leave one after the other (~0.13 us
                    // each), and with every CTA starting at rank 0 the high ranks had their h 1-2 us after the low ones
                    const int peer = (j + 1 + (et >> 1)) & (CS - 1);
                    const uint32_t src = sH + (et & 1) * h_half + off * 128;
                    bulk_copy_to_peer(map_to_rank(src, peer), src, (uint32_t)nj * 128u, map_to_rank(h_arr(j), peer));
                }
                if (et == 0 && i == 0) {
                    const long long e8 = RM_CLK();
                    RM_TR(item, 15, 0);
                    RM_PS(item, 3);
                    RM_PC(item, 16, e1 - e0); RM_PC(item, 17, e2 - e1); RM_PC(item, 18, e3 - e2); RM_PC(item, 19, e4 - e3);
                    RM_PC(item, 20, e5 - e4); RM_PC(item, 21, e6 - e5); RM_PC(item, 22, e7 - e6); RM_PC(item, 23, e8 - e7);
                }
            }
            if (stop) break;
            // Eq. 4, update step: the layer's output also holds gate * y_a.  The token rows c, c + NC, ... are this cluster's
            // share of that term, the columns of slice j this CTA's; it is added next to the CTA's own partial sums.
            const bool upd = EQ4 && anchor_mode == RM_ANCHOR_UPDATE;
            const bool ext = item_ext(env, l);
            const int* rctr = a.per_item ? a.sync + SYNC_RITEM + item : a.sync + SYNC_READ + b;
            const int rtarget = a.per_item ? n_ctas : a.sync_base[b] + n_ctas * (l + 1);
            if (run.ntiles == 0 && upd) {
                // no tiles, yet rows to add to: the same order of events as for a CTA with tiles (see the arrival below)
                if (et == 0 && !gave_up) {
                    if (!a.per_item && l > 0)
                        gave_up = counter_wait_slow(a.sync + b, a.sync_base[b] + n_ctas * l, __LINE__, sAbort, a.sync, a.status);
                    red_release_gpu(const_cast<int*>(rctr), 1);
                    if (!gave_up) gave_up = counter_wait_slow(rctr, rtarget, __LINE__, sAbort, a.sync, a.status);
                    if (l == 0 && pre && !gave_up)                 // r holds its copy of r_in
                        gave_up = counter_wait_slow(a.sync + SYNC_COPY + b, a.copy_base[b] + pre, __LINE__, sAbort, a.sync, a.status);
                }
                stop = named_barrier_or(1, 256, gave_up || *sAbort);
            }
            if (run.ntiles > 0) {
                // the item's down products are complete: add this CTA's [T x H/8] part to the residual stream
                const int d2b = ND2 == 2 ? (ni & 1) : 0, nu = ND2 == 2 ? (ni >> 1) : ni;
                ++ni;
                // The adds below go into the rows that every cluster has read for this item's normalisation.  Nothing else
                // orders a slower cluster's reads before them: wait for the count of the CTAs that have read.  (The
                // load is issued before the wait for the products, so its round trip is over by then.)
                const int rseen = lane == 0 && !ext ? ld_acquire_gpu(rctr) : rtarget;
                WAIT(d2_full(d2b), nu & 1);
                tc_fence_after();
                if (et == 0) RM_PS(item, 5);
                if (rseen < rtarget && !gave_up) gave_up = counter_wait_slow(rctr, rtarget, __LINE__, sAbort, a.sync, a.status);
                __syncwarp();
                if (l == 0 && pre) {
                    // r has to hold its copy of r_in before anything is added to it
                    if (lane == 0 && !gave_up) {
                        bool ok = false;
                        for (uint32_t w8 = 0; w8 < (1u << 21); ++w8) {
                            if (ld_acquire_gpu(a.sync + SYNC_COPY + b) >= a.copy_base[b] + pre) { ok = true; break; }
                            if ((w8 & 255u) == 255u && (*sAbort || ld_acquire_gpu(a.sync + SYNC_ABORT))) break;
                        }
                        if (!ok) { if (!*sAbort && !ld_acquire_gpu(a.sync + SYNC_ABORT)) timed_out(__LINE__); gave_up = true; *sAbort = 1; }
                    }
                    __syncwarp();
                }
                const size_t col0 = (size_t)j * HS8 + q4 * 32 + lane;
                float* rb = a.r + (size_t)b * T * H + col0;
                // Eq. 4: the sum is scaled by the output gate of its column on the way into r; the anchor step also
                // accumulates the sum as it is into y_a (cleared by the host before the launch)
                float gt0 = 1.f, gt1 = 1.f;
                if (EQ4 && a.gate) {
                    const float* gp = a.gate + ((size_t)l * B + b) * H + col0;
                    gt0 = __ldg(gp);
                    if (NMB == 2) gt1 = __ldg(gp + 128);
                }
                float* yb = EQ4 && anchor_mode == RM_ANCHOR_WRITE ? a.y_anchor + ((size_t)l * B + b) * T * H + col0 : nullptr;
                // (rolled loops over 8 token columns at a time: this code runs once per layer, and the smaller it is the
                // less of the other roles' loops it pushes out of the instruction cache)
#pragma unroll 1
                for (int q8 = 0; q8 < NMB * 4; ++q8) {
                    const int mb = q8 >> 2, c8 = (q8 & 3) * 8;
                    float hi[8], lo[8];
                    const uint32_t col = tmem + G::D2_COL + d2b * (2 * NTOK) + mb * (2 * NTOK) + ch * 32 + c8 + ((uint32_t)(q4 * 32) << 16);
                    tmem_ld8(col, hi);
                    tmem_ld8(col + NTOK, lo);
                    const size_t o = (size_t)(ch * 32 + c8) * H + mb * 128;
                    const float gt = EQ4 ? (mb ? gt1 : gt0) : 1.f;
#pragma unroll
                    for (int r = 0; r < 8; ++r)
                        if (ch * 32 + c8 + r < T) {
                            const float y = hi[r] + lo[r];
                            red_add_f32(rb + o + (size_t)r * H, EQ4 ? gt * y : y);
                            if (EQ4 && yb) red_add_f32(yb + o + (size_t)r * H, y);
                        }
                }
                tc_fence_before();
                mbar_arrive(d2_empty(d2b));
                if (et == 0) RM_PS(item, 6);
            }
            if (upd && !stop) {
                const int nrows = c < T ? (T - c + NC - 1) / NC : 0;
                const float* ya = a.y_anchor + ((size_t)l * B + b) * T * H + (size_t)j * HS8;
                const float* gp = a.gate ? a.gate + ((size_t)l * B + b) * H + (size_t)j * HS8 : nullptr;
                float* rr = a.r + (size_t)b * T * H + (size_t)j * HS8;
                for (int e = et; e < nrows * HS8; e += 256) {
                    const int ri = e / HS8, cc = e - ri * HS8;
                    const size_t o = (size_t)(c + ri * NC) * H + cc;
                    red_add_f32(rr + o, (gp ? __ldg(gp + cc) : 1.f) * __ldcg(ya + o));
                }
            }
            // no fence per thread: the barrier orders every thread's adds before thread 0's release on the counter
            // below, and a release is cumulative (the pattern of a grid-wide barrier: sync, then one thread fences)
            if (run.ntiles > 0 || upd) stop = named_barrier_or(1, 256, gave_up || *sAbort);
            if (et == 0) {
                // The episode's counter adds up the arrivals of all layers, and "n_ctas (l + 1) arrivals" means "every CTA has
                // added its part of layer l" only if nobody arrives for layer l before every CTA has arrived for layer l - 1.
                // A CTA with tiles in layer l has waited for exactly that before normalising; a CTA whose cluster has none
                // (lists shorter than the number of clusters) would otherwise run through its empty layers at once, and its
                // early arrivals would stand in for a slower CTA's.
                const bool empty = run.ntiles == 0 && !upd;
                if (empty && !a.per_item && l > 0 && !gave_up)
                    gave_up = counter_wait_slow(a.sync + b, a.sync_base[b] + n_ctas * l, __LINE__, sAbort, a.sync, a.status);
                // (CTAs that have not normalised this item -- no tiles, or x from the caller -- count as readers here)
                if (empty || (ext && run.ntiles > 0)) red_release_gpu(const_cast<int*>(rctr), 1);
                red_release_gpu(a.per_item ? a.sync + SYNC_ITEM + item : a.sync + b, 1);
                RM_PS(item, 7);
            }
        }
    }
#undef WAIT
    tc_fence_before();
    __syncthreads();
    if (*sAbort) {
        // a wait gave up somewhere: copies into this CTA's shared memory (x blocks, peers' h rows) may still be in flight
        // although nobody waits for them any more.  They land within microseconds; idle for longer than that.
        for (int i = 0; i < 64; ++i) __nanosleep(4000);
        __syncthreads();
    }
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
    auto kern = step_kernel<HS8, false>;
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

template <int HS8, bool EQ4>
int launch(rm_ctx* ctx, const PArgs& a, const CUtensorMap& tmXext, int n_clusters, cudaStream_t s) {
    static rm_smem_configured configured = {};
    if (!configured.covers(ctx->device, Geo<HS8>::TOTAL)) {
        RM_CUDA_TRY(cudaFuncSetAttribute(step_kernel<HS8, EQ4>, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<HS8>::TOTAL));
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
    RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, step_kernel<HS8, EQ4>, a, tmXext));
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
    return (H == 1024 || H == 2048) && T >= 1 && T <= NTOK && B >= 1 && B <= MAXB && ctx->g.L <= MAXL && ctx->g.L * B <= MAX_ITEMS &&
           ctx->persist_clusters > 0 && encode_fn() != nullptr;
}

size_t rm_persist_workspace_bytes(const rm_ctx* ctx) {
    if (ctx->persist_clusters <= 0) return 0;
    return SYNC_BYTES + (size_t)ctx->persist_clusters * 2 * NTOK * ctx->g.H * sizeof(__nv_bfloat16);
}

int rm_persist_debug_stamps(long long* host_out, int n) {
#ifdef RM_PHASE_TIMING
    if (n > 64 * 128 * 32) n = 64 * 128 * 32;
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
    a.r_in = sa.r_in ? sa.r_in : sa.r;
    a.sync = reinterpret_cast<int*>(ws);
    a.xbuf = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(ws) + SYNC_BYTES);
    a.per_item = sa.B > 1 ? 1 : 0;
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
    a.pf_bytes = ctx->persist_prefetch_kb * 1024;
    int nc = ctx->persist_clusters;
    if (ctx->max_clusters_override > 0 && ctx->max_clusters_override < nc) nc = ctx->max_clusters_override;
    // the caller's x (single-layer entry) as a tensor map; otherwise any valid map (the kernel does not use it): one over
    // the workspace, made once per workspace
    if (!sa.x_ext && ctx->persist_xbuf != a.xbuf) {
        const int rc = make_x_map(reinterpret_cast<CUtensorMap*>(ctx->persist_tm), a.xbuf, (uint64_t)NTOK, (uint64_t)g.H);
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
    int nc_ctas = nc * CS;
    const int pre = a.r_in != a.r ? CS : 0;
    // The arrival counters live in the workspace and only ever count up; the host keeps their values.  They are cleared
    // when the workspace is new to this context, after a launch whose status was not clean (its count is unknown), and
    // long before they could wrap.
    bool reset = ctx->persist_sync != a.sync || ctx->persist_sync_dirty || a.per_item;
    for (int b = 0; b < MAXB; ++b) reset = reset || ctx->persist_sync_base[b] > (1 << 30);
    if (reset) {
        RM_CUDA_TRY(cudaMemsetAsync(a.sync, 0, a.per_item ? SYNC_BYTES : 256, s));
        for (int b = 0; b < MAXB; ++b) ctx->persist_sync_base[b] = ctx->persist_copy_base[b] = 0;
        ctx->persist_sync = a.sync;
        ctx->persist_sync_dirty = 0;
    }
    for (int b = 0; b < MAXB; ++b) { a.sync_base[b] = ctx->persist_sync_base[b]; a.copy_base[b] = ctx->persist_copy_base[b]; }
    for (int b = 0; b < sa.B; ++b) { ctx->persist_sync_base[b] += nc_ctas * sa.L; ctx->persist_copy_base[b] += pre; }
    // (the instantiation without Eq. 4 and gate is the one the plain steps run: it carries none of their code)
    const bool eq4 = sa.anchor_mode != RM_ANCHOR_NONE || sa.gate != nullptr;
    a.anchor_mode = sa.anchor_mode;
    a.y_anchor = sa.y_anchor;
    a.h_anchor = sa.h_anchor;
    a.h_stride = sa.h_stride;
    a.gate = sa.gate;
    // the anchor step's sums are accumulated by the CTAs' atomics: start them from zero
    if (sa.anchor_mode == RM_ANCHOR_WRITE)
        RM_CUDA_TRY(cudaMemsetAsync(sa.y_anchor, 0, (size_t)sa.L * sa.B * sa.T * g.H * sizeof(float), s));
    const int rc = g.H == 1024 ? (eq4 ? launch<128, true>(ctx, a, tm_ext, nc, s) : launch<128, false>(ctx, a, tm_ext, nc, s))
                               : (eq4 ? launch<256, true>(ctx, a, tm_ext, nc, s) : launch<256, false>(ctx, a, tm_ext, nc, s));
    if (rc != RM_OK) ctx->persist_sync_dirty = 1;               // nothing ran: the counters are behind the host's count
    return rc;
}
