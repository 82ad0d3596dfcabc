// Gather-read microbenchmark: the access pattern of the layer kernels' loaders and nothing else.  For a list of
// neurons, CTA (group g, slice j) reads the 3*Hs*2-byte piece j of every neuron of tiles g, g + G, ... with 16-byte
// cp.async into two shared-memory stages and throws the data away.  Timed by the caller, it says how fast this list
// can leave HBM at all with this pattern -- the ceiling the layer kernels are measured against besides the copy
// bandwidth.
#include "rm_common.cuh"
#include "rm_sm100.cuh"

using namespace sm100;

namespace {

constexpr int GT = 128;                // threads per CTA
constexpr int GNT = 64;                // neurons per tile

__global__ void __launch_bounds__(GT) gather_read_kernel(const __nv_bfloat16* __restrict__ packed,
                                                         const int32_t* __restrict__ idx, const int32_t* __restrict__ count,
                                                         int64_t cap, int H, int I, int* status) {
    extern __shared__ unsigned char smem[];
    const int j = blockIdx.x & 7, g = blockIdx.x >> 3, G = gridDim.x >> 3;
    const int Hs = H / 8, chunks = 3 * Hs * 2 / 16;        // 16-byte chunks per piece
    const uint32_t base = (smem_u32(smem) + 127u) & ~127u;
    const int stage_bytes = GNT * chunks * 16;
    int c = idx ? *count : I;
    if (c < 0 || c > cap || c > I) {
        if (blockIdx.x == 0 && threadIdx.x == 0) rm_set_status(status, RM_ERR_INDEX);
        c = c < 0 ? 0 : (int)(cap < (int64_t)I ? cap : (int64_t)I);
    }
    const int tiles = (c + GNT - 1) / GNT;
    int k = 0;
    for (int t = g; t < tiles; t += G, ++k) {
        const uint32_t st = base + (k & 1) * stage_bytes;
        if (k >= 2) cp_async_wait<1>();                    // the stage's previous tile has landed
        for (int e = threadIdx.x; e < GNT * chunks; e += GT) {
            const int q = e / chunks, ch = e - q * chunks;
            const int p = t * GNT + q;
            int n = p < c ? (idx ? idx[p] : p) : -1;
            if (n >= I) n = -1;
            cp_async16(st + e * 16, packed + (size_t)(n < 0 ? 0 : n) * 3 * H + (size_t)j * 3 * Hs + ch * 8, n >= 0);
        }
        cp_async_commit();
    }
    cp_async_wait<0>();
}

}  // namespace

int rm_launch_gather_read(rm_ctx* ctx, const void* packed, const int32_t* idx, const int32_t* count, int64_t cap,
                          cudaStream_t s) {
    const rm_geom& g = ctx->g;
    if (g.H % 64 != 0) return RM_ERR_UNSUPPORTED;
    const int smem = 2 * GNT * 3 * g.Hs * 2 + 128;
    if (smem > 200 * 1024) return RM_ERR_UNSUPPORTED;
    static rm_smem_configured configured = {};
    if (!configured.covers(ctx->device, smem)) {
        RM_CUDA_TRY(cudaFuncSetAttribute(gather_read_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        configured.set(ctx->device, smem);
    }
    const int groups = ctx->sm_count >= 8 ? ctx->sm_count / 8 : 1;             // 18 groups of 8 CTAs on 148 SMs
    gather_read_kernel<<<groups * 8, GT, smem, s>>>(static_cast<const __nv_bfloat16*>(packed), idx, count, cap, g.H, g.I,
                                                    ctx->d_status);
    ctx->launches++;
    RM_CUDA_TRY(cudaGetLastError());
    return RM_OK;
}
