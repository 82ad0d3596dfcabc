// rm_pack_weights: one-off repacking of a layer into the neuron-major layout (see rm_geom in rm_common.cuh),
// and the per-neuron down-projection column norm ||Wd[:,n]||_2, the weight factor of Eq. 1.
#include "rm_common.cuh"

namespace {

// One CTA per (neuron tile of 32, column slice).  Gate / up pieces are straight row copies; the down piece is a
// 32 x Hs transpose staged through shared memory so that both the global reads (along n) and the global writes
// (along the column) are coalesced.
__global__ void __launch_bounds__(256) pack_kernel(const __nv_bfloat16* __restrict__ Wg,
                                                   const __nv_bfloat16* __restrict__ Wu,
                                                   const __nv_bfloat16* __restrict__ Wd,
                                                   __nv_bfloat16* __restrict__ out, rm_geom g) {
    extern __shared__ __nv_bfloat16 tile[];                 // [Hs][33]
    const int n0 = blockIdx.x * 32;
    const int j = blockIdx.y;
    const int Hs = g.Hs;
    // gate and up
    for (int e = threadIdx.x; e < 32 * Hs; e += blockDim.x) {
        int q = e / Hs, kk = e - q * Hs;
        int n = n0 + q;
        if (n < g.I) {
            out[g.off(n, 0, j * Hs + kk)] = Wg[(size_t)n * g.H + j * Hs + kk];
            out[g.off(n, 1, j * Hs + kk)] = Wu[(size_t)n * g.H + j * Hs + kk];
        }
    }
    // down: read Wd[c, n0..n0+31] (contiguous in n), write out[n][slice j][down][c]
    for (int e = threadIdx.x; e < 32 * Hs; e += blockDim.x) {
        int kk = e >> 5, q = e & 31;
        int n = n0 + q;
        tile[kk * 33 + q] = n < g.I ? Wd[(size_t)(j * Hs + kk) * g.I + n] : __float2bfloat16(0.0f);
    }
    __syncthreads();
    for (int e = threadIdx.x; e < 32 * Hs; e += blockDim.x) {
        int q = e / Hs, kk = e - q * Hs;
        int n = n0 + q;
        if (n < g.I) out[g.off(n, 2, j * Hs + kk)] = tile[kk * 33 + q];
    }
}

__global__ void __launch_bounds__(256) colnorm_kernel(const __nv_bfloat16* __restrict__ Wd, float* __restrict__ out,
                                                      int H, int I) {
    int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= I) return;
    float s = 0.0f;
    for (int c = 0; c < H; ++c) {
        float v = __bfloat162float(Wd[(size_t)c * I + n]);
        s = fmaf(v, v, s);
    }
    out[n] = sqrtf(s);
}

// Compact copy of the listed neurons' packed rows: out row p = packed row idx[p], p < count (rows up to the next
// multiple of 64 are cleared, later rows are left alone).  One warp per row
// (3H bf16, contiguous in both buffers), 16 bytes per lane and iteration.
__global__ void __launch_bounds__(256) gather_rows_kernel(const uint4* __restrict__ packed, const int32_t* __restrict__ idx,
                                                          const int32_t* __restrict__ count, int64_t cap,
                                                          uint4* __restrict__ out, int row_u4, int I, int* status) {
    const int p = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    int c = *count;
    if (c < 0 || c > cap || c > I) {
        if (blockIdx.x == 0 && threadIdx.x == 0) rm_set_status(status, RM_ERR_INDEX);
        c = c < 0 ? 0 : (int)(cap < (int64_t)I ? cap : (int64_t)I);
    }
    if (p >= c) {
        // the rest of the last 64-neuron tile is zero-filled: kernels that fetch a compact layer in whole-tile boxes
        // multiply those rows by h = 0, which must not meet a NaN left in the buffer
        const int64_t rows = cap < (int64_t)I ? cap : (int64_t)I;
        if (p < ((c + 63) & ~63) && p < rows)
            for (int e = lane; e < row_u4; e += 32) out[(size_t)p * row_u4 + e] = make_uint4(0, 0, 0, 0);
        return;
    }
    const int n = idx[p];
    if (n < 0 || n >= I) {
        if (lane == 0) rm_set_status(status, RM_ERR_INDEX);
        for (int e = lane; e < row_u4; e += 32) out[(size_t)p * row_u4 + e] = make_uint4(0, 0, 0, 0);
        return;
    }
    const uint4* src = packed + (size_t)n * row_u4;
    for (int e = lane; e < row_u4; e += 32) out[(size_t)p * row_u4 + e] = src[e];
}

}  // namespace

int rm_launch_gather_rows(rm_ctx* ctx, const void* packed, const int32_t* idx, const int32_t* count, int64_t cap,
                          void* out, cudaStream_t s) {
    const rm_geom& g = ctx->g;
    const int row_u4 = 3 * g.H * (int)sizeof(__nv_bfloat16) / 16;
    const int64_t rows = cap < (int64_t)g.I ? cap : (int64_t)g.I;
    if (rows <= 0) return RM_OK;
    gather_rows_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, s>>>(static_cast<const uint4*>(packed), idx, count, cap,
                                                                 static_cast<uint4*>(out), row_u4, g.I, ctx->d_status);
    ctx->launches++;
    RM_CUDA_TRY(cudaGetLastError());
    return RM_OK;
}

int rm_launch_pack(rm_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, void* packed, float* colnorm,
                   cudaStream_t s) {
    const rm_geom& g = ctx->g;
    dim3 grid((g.I + 31) / 32, RM_NS);
    size_t smem = (size_t)g.Hs * 33 * sizeof(__nv_bfloat16);
    if (smem > 48 * 1024)
        RM_CUDA_TRY(cudaFuncSetAttribute(pack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    pack_kernel<<<grid, 256, smem, s>>>(static_cast<const __nv_bfloat16*>(Wg), static_cast<const __nv_bfloat16*>(Wu),
                                        static_cast<const __nv_bfloat16*>(Wd), static_cast<__nv_bfloat16*>(packed), g);
    ctx->launches++;
    RM_CUDA_TRY(cudaGetLastError());
    if (colnorm) {
        colnorm_kernel<<<(g.I + 255) / 256, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(Wd), colnorm, g.H, g.I);
        ctx->launches++;
        RM_CUDA_TRY(cudaGetLastError());
    }
    return RM_OK;
}
