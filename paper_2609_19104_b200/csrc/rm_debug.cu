// Measurement and test aids (not part of the method).
//
// gather_read_kernel: the practical ceiling of reading the listed neurons' packed rows and nothing else.  One CTA per SM;
// CTA c takes list positions c, c + G, ... of every layer handed to it and pulls each neuron's whole 6*H-byte row into a
// ring of shared-memory stages with 16-byte cp.async (the instruction the layer kernels gather with), 12 rows in
// flight, then throws the data away.  One launch covers one layer or a whole step's layers back to back.  Timed by the
// caller it says how fast these lists can leave HBM at all.
//
// wait_timeout_kernel: one CTA waits on an mbarrier that nobody arrives at, with a small poll budget, records
// RM_ERR_TIMEOUT with the source line of the wait like the layer kernels' bounded waits do, and returns.
#include "rm_common.cuh"
#include "rm_sm100.cuh"

using namespace sm100;

namespace {

constexpr int GT = 256;                // threads per CTA
constexpr int DEPTH = 12;              // rows in flight per CTA
constexpr int MAXL_DBG = 64;

struct GatherArgs {
    const __nv_bfloat16* packed[MAXL_DBG];
    const int32_t* idx;                // list of layer l at idx + l * stride; NULL: every neuron
    const int32_t* count;              // count of layer l at count[l]
    int64_t stride, cap;
    int L, H, I;
    int* status;
};

constexpr int MAX_ROWS_PER_CTA = 512;  // list positions one CTA takes per layer (I / CTAs, rounded up)

__global__ void __launch_bounds__(GT) gather_read_kernel(const __grid_constant__ GatherArgs a) {
    extern __shared__ unsigned char smem[];
    __shared__ int ids[2][MAX_ROWS_PER_CTA];
    __shared__ int cnts[2];
    const uint32_t base = (smem_u32(smem) + 127u) & ~127u;
    const int row_bytes = 6 * a.H, pieces = row_bytes / 16;
    // the neuron ids of this CTA's list positions, one layer ahead of the reads (an id fetched right before its row
    // would put an L2 round trip in front of every row)
    auto fetch_ids = [&](int l) {
        int c = a.idx ? a.count[l] : a.I;
        if (c < 0 || c > a.cap || c > a.I) {
            if (blockIdx.x == 0 && threadIdx.x == 0) rm_set_status(a.status, RM_ERR_INDEX);
            c = c < 0 ? 0 : (int)(a.cap < (int64_t)a.I ? a.cap : (int64_t)a.I);
        }
        const int32_t* list = a.idx ? a.idx + (size_t)l * a.stride : nullptr;
        const int mine = c > (int)blockIdx.x ? (c - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
        for (int k = threadIdx.x; k < mine && k < MAX_ROWS_PER_CTA; k += GT) {
            const int p = blockIdx.x + k * gridDim.x;
            int n = list ? list[p] : p;
            ids[l & 1][k] = (n < 0 || n >= a.I) ? -1 : n;
        }
        if (threadIdx.x == 0) cnts[l & 1] = mine < MAX_ROWS_PER_CTA ? mine : MAX_ROWS_PER_CTA;
    };
    fetch_ids(0);
    __syncthreads();
    int k = 0;
    for (int l = 0; l < a.L; ++l) {
        if (l + 1 < a.L) fetch_ids(l + 1);
        const int mine = cnts[l & 1];
        for (int r = 0; r < mine; ++r, ++k) {
            const int n = ids[l & 1][r];
            const uint32_t st = base + (k % DEPTH) * row_bytes;
            if (k >= DEPTH) cp_async_wait<DEPTH - 1>();        // the stage's previous row has landed
            const __nv_bfloat16* src = a.packed[l] + (size_t)(n < 0 ? 0 : n) * 3 * a.H;
            for (int e = threadIdx.x; e < pieces; e += GT) cp_async16(st + e * 16, src + e * 8, n >= 0);
            cp_async_commit();
        }
        __syncthreads();
    }
    cp_async_wait<0>();
}

__global__ void __launch_bounds__(32) wait_timeout_kernel(int* status, unsigned polls) {
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        fence_mbar_init();
        // nobody arrives: the wait runs out of its budget, records where it gave up, and the kernel returns
        if (!mbar_wait(b, 0, polls)) rm_set_status_at(status, RM_ERR_TIMEOUT, (__LINE__ << 12) | (int)(blockIdx.x & 0xfffu));
    }
}

int launch_gather(rm_ctx* ctx, const GatherArgs& a, cudaStream_t s) {
    const rm_geom& g = ctx->g;
    if (g.H % 64 != 0) return RM_ERR_UNSUPPORTED;
    const int smem = DEPTH * 6 * g.H + 128;
    if (smem > 227 * 1024) return RM_ERR_UNSUPPORTED;
    static rm_smem_configured configured = {};
    if (!configured.covers(ctx->device, smem)) {
        RM_CUDA_TRY(cudaFuncSetAttribute(gather_read_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        configured.set(ctx->device, smem);
    }
    gather_read_kernel<<<ctx->sm_count > 0 ? ctx->sm_count : 148, GT, smem, s>>>(a);
    ctx->launches++;
    RM_CUDA_TRY(cudaGetLastError());
    return RM_OK;
}

}  // namespace

int rm_launch_gather_read(rm_ctx* ctx, const void* packed, const int32_t* idx, const int32_t* count, int64_t cap,
                          cudaStream_t s) {
    GatherArgs a{};
    a.packed[0] = static_cast<const __nv_bfloat16*>(packed);
    a.idx = idx;
    a.count = count;
    a.stride = 0;
    a.cap = cap;
    a.L = 1;
    a.H = ctx->g.H;
    a.I = ctx->g.I;
    a.status = ctx->d_status;
    return launch_gather(ctx, a, s);
}

int rm_launch_gather_read_step(rm_ctx* ctx, const void* const* packed_layers, const int32_t* idx, const int32_t* count,
                               int64_t stride, cudaStream_t s) {
    if (ctx->g.L > MAXL_DBG) return RM_ERR_UNSUPPORTED;
    GatherArgs a{};
    for (int l = 0; l < ctx->g.L; ++l) a.packed[l] = static_cast<const __nv_bfloat16*>(packed_layers[l]);
    a.idx = idx;
    a.count = count;
    a.stride = stride;
    a.cap = idx ? stride : ctx->g.I;
    a.L = ctx->g.L;
    a.H = ctx->g.H;
    a.I = ctx->g.I;
    a.status = ctx->d_status;
    return launch_gather(ctx, a, s);
}

int rm_launch_wait_timeout(rm_ctx* ctx, unsigned polls, cudaStream_t s) {
    wait_timeout_kernel<<<1, 32, 0, s>>>(ctx->d_status, polls);
    ctx->launches++;
    RM_CUDA_TRY(cudaGetLastError());
    return RM_OK;
}
