// rm_mask_compact: important-neuron selection and stream compaction, one CTA per list.
//
// A list is one (layer, episode) pair.  Every record of the list is reduced to a per-neuron flag by the chosen
// rule (boolean, score > threshold, or the k largest scores with ties going to the lower index -- the ranking of
// Eq. 1's contribution scores), the flags are combined by a vote, and the surviving neurons are written in
// ascending order with warp-ballot / popc prefix sums.  Exact top-k uses a 4-pass, 8-bit radix select on
// order-preserving integer keys, so the result is the unique set a full sort with (score descending, index
// ascending) would give.
#include "rm_common.cuh"

namespace {

constexpr int MASK_THREADS = 1024;
constexpr int MASK_MAX_RECORDS = 16;

struct MaskParams {
    const void* rec[MASK_MAX_RECORDS];
    int W, kind, reduce, k, min_votes, scale_per_list, I;
    float threshold;
    const float* scale;
    int64_t stride;
    int32_t* idx_out;
    int32_t* count_out;
    int* status;
};

struct MaskShared {
    unsigned hist[256];
    int warp_tot[32];
    int scan_total;
    unsigned sel_prefix;       // radix-select state
    int sel_remaining;
};

// order-preserving key: larger float -> larger key; -0 == +0; NaN below everything
__device__ __forceinline__ unsigned key_of(float s) {
    if (s != s) return 0u;
    if (s == 0.0f) s = 0.0f;                       // folds -0 into +0
    unsigned u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ float load_score(const MaskParams& p, int w, int list, int n) {
    float s = static_cast<const float*>(p.rec[w])[(size_t)list * p.I + n];
    if (p.scale) s *= p.scale[(p.scale_per_list ? (size_t)list * p.I : 0) + n];
    return s;
}

// Exclusive rank of `pred` among the CTA's threads in thread order, and the CTA total (all threads get both).
__device__ __forceinline__ int block_rank(bool pred, MaskShared& sh, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned b = __ballot_sync(0xffffffffu, pred);
    int in_warp = __popc(b & ((1u << lane) - 1u));
    if (lane == 0) sh.warp_tot[warp] = __popc(b);
    __syncthreads();
    if (warp == 0) {
        int v = sh.warp_tot[lane];
        int incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            int o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        sh.warp_tot[lane] = incl - v;              // exclusive prefix of warp totals
        if (lane == 31) sh.scan_total = incl;
    }
    __syncthreads();
    int r = sh.warp_tot[warp] + in_warp;
    total = sh.scan_total;
    __syncthreads();                               // warp_tot / scan_total may be rewritten by the next call
    return r;
}

// Radix select over the elements for which valid(n) holds: finds the key of the kk-th largest element
// (1 <= kk <= number of valid elements) and how many elements equal to that key belong to the top kk.
template <class KeyFn, class ValidFn>
__device__ void select_kth(int I, int kk, KeyFn key, ValidFn valid, MaskShared& sh, unsigned& kth, int& take_equal) {
    if (threadIdx.x == 0) { sh.sel_prefix = 0u; sh.sel_remaining = kk; }
    unsigned mask = 0u;
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (threadIdx.x < 256) sh.hist[threadIdx.x] = 0u;
        __syncthreads();
        const unsigned prefix = sh.sel_prefix;
        for (int n = threadIdx.x; n < I; n += MASK_THREADS) {
            if (!valid(n)) continue;
            unsigned kv = key(n);
            if ((kv & mask) == prefix) atomicAdd(&sh.hist[(kv >> shift) & 0xFFu], 1u);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // lane l owns bins [8l, 8l+8); walk from the highest bin down
            const int lane = threadIdx.x;
            unsigned c[8], mine = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) { c[i] = sh.hist[lane * 8 + i]; mine += c[i]; }
            unsigned above = 0u;                    // elements in bins of higher lanes
            unsigned run = mine;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                unsigned o = __shfl_down_sync(0xffffffffu, run, d);
                if (lane + d < 32) run += o;
            }
            above = run - mine;                     // suffix sum excluding this lane
            const unsigned rem = (unsigned)sh.sel_remaining;
            __syncwarp();                           // every lane has read `rem` before one lane rewrites it
            if (above < rem && rem <= above + mine) {
                unsigned acc = above;
#pragma unroll
                for (int i = 7; i >= 0; --i) {
                    if (acc < rem && rem <= acc + c[i]) {
                        sh.sel_prefix = prefix | ((unsigned)(lane * 8 + i) << shift);
                        sh.sel_remaining = (int)(rem - acc);
                    }
                    acc += c[i];
                }
            }
        }
        mask |= 0xFFu << shift;
        __syncthreads();
    }
    kth = sh.sel_prefix;
    take_equal = sh.sel_remaining;
    __syncthreads();
}

// Flags the top-kk valid elements into out[n] via op(n, flag); ties at the k-th key go to the lower index.
template <class KeyFn, class ValidFn, class OutFn>
__device__ void flag_topk(int I, int k, int n_valid, KeyFn key, ValidFn valid, OutFn out, MaskShared& sh) {
    const int kk = k < n_valid ? k : n_valid;
    if (kk <= 0) {
        for (int n = threadIdx.x; n < I; n += MASK_THREADS) out(n, false);
        __syncthreads();
        return;
    }
    if (kk >= n_valid) {
        for (int n = threadIdx.x; n < I; n += MASK_THREADS) out(n, valid(n));
        __syncthreads();
        return;
    }
    unsigned kth; int take_equal;
    select_kth(I, kk, key, valid, sh, kth, take_equal);
    int eq_before = 0;
    for (int base = 0; base < I; base += MASK_THREADS) {
        const int n = base + threadIdx.x;
        bool v = n < I && valid(n);
        unsigned kv = v ? key(n) : 0u;
        bool eq = v && kv == kth, gt = v && kv > kth;
        int total;
        int r = block_rank(eq, sh, total);
        if (n < I) out(n, gt || (eq && eq_before + r < take_equal));
        eq_before += total;
    }
    __syncthreads();
}

__global__ void __launch_bounds__(MASK_THREADS) mask_compact_kernel(MaskParams p) {
    extern __shared__ __align__(16) unsigned char votes[];      // [I]
    __shared__ MaskShared sh;
    const int list = blockIdx.x;
    const int I = p.I;

    for (int n = threadIdx.x; n < I; n += MASK_THREADS) votes[n] = 0;
    // programmatic dependent launch: a kernel launched behind this one may start its prologue now; the records read
    // below may come from the kernel in front of this one
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __syncthreads();

    auto all_valid = [](int) { return true; };
    auto add_vote = [&](int n, bool f) { votes[n] += f ? 1 : 0; };

    for (int w = 0; w < p.W; ++w) {
        if (p.kind == RM_SRC_BOOL_U8) {
            const unsigned char* m = static_cast<const unsigned char*>(p.rec[w]) + (size_t)list * I;
            for (int n = threadIdx.x; n < I; n += MASK_THREADS) votes[n] += m[n] != 0 ? 1 : 0;
            __syncthreads();
        } else if (p.reduce == RM_REDUCE_THRESHOLD) {
            for (int n = threadIdx.x; n < I; n += MASK_THREADS)
                votes[n] += load_score(p, w, list, n) > p.threshold ? 1 : 0;
            __syncthreads();
        } else {                                    // TOPK, and the per-record stage of GROUP
            auto key = [&](int n) { return key_of(load_score(p, w, list, n)); };
            flag_topk(I, p.k, I, key, all_valid, add_vote, sh);
        }
    }

    int need = p.min_votes;
    if (p.reduce == RM_REDUCE_GROUP) {
        // rank the union of the per-record sets by the summed score and keep the top k; bit 7 of votes[n]
        // marks "kept" (vote counts are at most 16, so it is free)
        __shared__ int s_union;
        if (threadIdx.x == 0) s_union = 0;
        __syncthreads();
        int mine = 0;
        for (int n = threadIdx.x; n < I; n += MASK_THREADS) mine += votes[n] != 0;
        if (mine) atomicAdd(&s_union, mine);
        __syncthreads();
        const int n_union = s_union;
        auto in_union = [&](int n) { return (votes[n] & 0x7F) != 0; };
        auto key = [&](int n) {
            float s = 0.0f;
            for (int w = 0; w < p.W; ++w) s += load_score(p, w, list, n);
            return key_of(s);
        };
        auto mark = [&](int n, bool f) { if (f) votes[n] |= 0x80; };
        flag_topk(I, p.k, n_union, key, in_union, mark, sh);
        need = 0x80;                                // kept <=> bit 7 set <=> value >= 128
    }

    // ordered compaction of { n : votes[n] >= need }
    int32_t* out = p.idx_out + (size_t)list * p.stride;
    int written = 0;
    bool overflow = false;
    for (int base = 0; base < I; base += MASK_THREADS) {
        const int n = base + threadIdx.x;
        bool keep = n < I && (int)votes[n] >= need;
        int total;
        int r = block_rank(keep, sh, total);
        if (keep) {
            int pos = written + r;
            if (pos < p.stride) out[pos] = n; else overflow = true;
        }
        written += total;
    }
    if (overflow) rm_set_status(p.status, RM_ERR_INDEX);
    if (threadIdx.x == 0) p.count_out[list] = written < p.stride ? written : (int)p.stride;
}

}  // namespace

int rm_launch_mask_compact(rm_ctx* ctx, const rm_mask_src* src, int32_t* idx_out, int32_t* count_out,
                           int64_t stride, cudaStream_t s) {
    MaskParams p{};
    for (int w = 0; w < src->n_records; ++w) p.rec[w] = src->records[w];
    p.W = src->n_records;
    p.kind = src->kind;
    p.reduce = src->reduce;
    p.k = src->k;
    p.min_votes = src->reduce == RM_REDUCE_GROUP ? 1 : src->min_votes;
    p.scale_per_list = src->scale_per_list;
    p.I = src->I;
    p.threshold = src->threshold;
    p.scale = src->scale;
    p.stride = stride;
    p.idx_out = idx_out;
    p.count_out = count_out;
    p.status = ctx->d_status;
    size_t smem = ((size_t)src->I + 15) & ~(size_t)15;
    if (smem > 200 * 1024) return RM_ERR_UNSUPPORTED;
    if (smem > 40 * 1024)
        RM_CUDA_TRY(cudaFuncSetAttribute(mask_compact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    if (src->n_lists > 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(src->n_lists);
        cfg.blockDim = dim3(MASK_THREADS);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = s;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        RM_CUDA_TRY(cudaLaunchKernelEx(&cfg, mask_compact_kernel, p));
        ctx->launches++;
    }
    return RM_OK;
}
