// Thin wrappers over the sm_100a instructions the fused layer kernel uses: tcgen05 (MMA into tensor memory,
// TMEM allocation and loads), mbarrier, cp.async, cluster barriers, distributed shared memory and programmatic
// dependent launch.  Every wait is bounded.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace sm100 {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---------------------------------------------------------------- cluster
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_count_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync() { cluster_arrive(); cluster_wait(); }

// address of the same shared-memory location in the CTA of rank `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t cta_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(cta_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t addr, float a, float b, float c, float d) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void st_cluster_v4u(uint32_t addr, uint4 v) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float a) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(a) : "memory");
}

// Asynchronous stores into a peer CTA's shared memory that also count their bytes on an mbarrier of that CTA
// (both addresses in the shared::cluster window, same CTA).  The receiver learns that the data has arrived by
// waiting on its own barrier; the sender needs no acknowledgement and no cluster-wide barrier.
__device__ __forceinline__ void st_async_v4(uint32_t addr, float a, float b, float c, float d, uint32_t mbar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d), "r"(mbar) : "memory");
}
__device__ __forceinline__ void st_async_v4u(uint32_t addr, uint4 v, uint32_t mbar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(mbar) : "memory");
}
__device__ __forceinline__ void st_async_f32(uint32_t addr, float a, uint32_t mbar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];"
                 ::"r"(addr), "f"(a), "r"(mbar) : "memory");
}

// Bulk copy from this CTA's shared memory into a peer's (size a multiple of 16 bytes, both 16-byte aligned); the
// bytes are counted on an mbarrier of the destination CTA.  Issued by one thread; the copy engine moves the data.
__device__ __forceinline__ void bulk_copy_to_peer(uint32_t dst_cluster_addr, uint32_t src_cta_addr, uint32_t bytes,
                                                  uint32_t mbar_cluster_addr) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster_addr), "r"(src_cta_addr), "r"(bytes), "r"(mbar_cluster_addr) : "memory");
}

// fire-and-forget vector add to global memory (16-byte aligned address)
__device__ __forceinline__ void red_add_f32(float* addr, float a) {
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(addr), "f"(a) : "memory");
}
__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// Bulk add of fp32 data from this CTA's shared memory into global memory by the copy engine: a contiguous piece
// (16-byte aligned on both sides, size a multiple of 16 bytes), or one box of a tiled tensor map (rows outside the
// tensor's extent are dropped; the innermost coordinate times 4 bytes must be a multiple of 16 and no coordinate may
// be negative).  The writer fences its shared-memory stores for the async proxy first; the issuing thread commits a
// group and waits for the group's reads before the source is reused or the CTA exits.
__device__ __forceinline__ void bulk_reduce_add_f32(float* dst, uint32_t src_cta_addr, uint32_t bytes) {
    asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;"
                 ::"l"(dst), "r"(src_cta_addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tensor_reduce_add_3d(const void* tensor_map, int x, int y, int z, uint32_t src_cta_addr) {
    asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(reinterpret_cast<uint64_t>(tensor_map)), "r"(x), "r"(y), "r"(z), "r"(src_cta_addr) : "memory");
}
// One box of a tiled tensor map into this CTA's shared memory; its bytes are counted on an mbarrier of this CTA.  The
// innermost coordinate times the element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tensor_map, int x, int y, uint32_t mbar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tensor_map)), "r"(x), "r"(y), "r"(mbar) : "memory");
}
// A contiguous piece of global memory (16-byte aligned, size a multiple of 16) into this CTA's shared memory; its bytes
// are counted on an mbarrier of this CTA.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t mbar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(mbar) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... until at most the newest group is still reading its source
__device__ __forceinline__ void bulk_wait_read_but_one() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }

// ---------------------------------------------------------------- programmatic dependent launch
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------- cp.async (16-byte gathers into swizzled tiles)
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    int sz = valid ? 16 : 0;       // src-size 0 writes 16 zero bytes
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// ask the copy engine to bring `bytes` (multiple of 16, 16-byte aligned) of global memory into L2
__device__ __forceinline__ void prefetch_l2(const void* p, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}
// arrive on an mbarrier (of this CTA) once all cp.async operations this thread has issued so far have landed; the
// arrival is one of the barrier's expected count (no increment)
__device__ __forceinline__ void cp_async_arrive_noinc(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// barrier among a subset of the CTA's warps (id 1..15; `count` threads, a multiple of 32)
__device__ __forceinline__ void named_barrier(int id, int count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
// make generic-proxy writes to shared memory visible to the async proxy (tcgen05.mma reads operands through it)
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
// the same for this CTA's shared memory only (cheaper; enough when the reader is this CTA's own copy engine or MMA)
// (restricted to global memory: for generic-proxy stores to global memory that a bulk copy reads afterwards)
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
// one arrival plus the number of bytes that asynchronous stores will deliver in this phase
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Non-blocking test of a phase (try_wait may suspend the thread for a while even when the phase is complete)
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Tests of several phases whose answers come back together: one test takes ~200 clocks to return even when the phase
// is long complete, and a thread that looks at each answer before it starts the next test pays that once per test.
// Bit i of the result: the phase with parity `parity` of the mbarrier at base + 8 i has completed (i < 8); bit 8: the
// phase with parity `parity_x` of the mbarrier `extra`.
__device__ __forceinline__ uint32_t mbar_test_wait_8_1(uint32_t base, uint32_t parity, uint32_t extra, uint32_t parity_x) {
    uint32_t m;
    asm volatile(
        "{\n\t.reg .pred p0, p1, p2, p3, p4, p5, p6, p7, p8;\n\t.reg .b32 t;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p8, [%3], %4;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p0, [%1], %2;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p1, [%1+8], %2;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p2, [%1+16], %2;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p3, [%1+24], %2;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p4, [%1+32], %2;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p5, [%1+40], %2;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p6, [%1+48], %2;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p7, [%1+56], %2;\n\t"
        "selp.u32 %0, 256, 0, p8;\n\t"
        "selp.u32 t, 1, 0, p0;\n\tor.b32 %0, %0, t;\n\t"
        "selp.u32 t, 2, 0, p1;\n\tor.b32 %0, %0, t;\n\t"
        "selp.u32 t, 4, 0, p2;\n\tor.b32 %0, %0, t;\n\t"
        "selp.u32 t, 8, 0, p3;\n\tor.b32 %0, %0, t;\n\t"
        "selp.u32 t, 16, 0, p4;\n\tor.b32 %0, %0, t;\n\t"
        "selp.u32 t, 32, 0, p5;\n\tor.b32 %0, %0, t;\n\t"
        "selp.u32 t, 64, 0, p6;\n\tor.b32 %0, %0, t;\n\t"
        "selp.u32 t, 128, 0, p7;\n\tor.b32 %0, %0, t;\n\t}"
        : "=&r"(m) : "r"(base), "r"(parity), "r"(extra), "r"(parity_x) : "memory");
    return m;
}
// The same for two phases: bit 0 for (a, parity_a), bit 1 for (b, parity_b)
__device__ __forceinline__ uint32_t mbar_test_wait_2(uint32_t a, uint32_t parity_a, uint32_t b, uint32_t parity_b) {
    uint32_t m;
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b32 t;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p0, [%1], %2;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p1, [%3], %4;\n\t"
        "selp.u32 %0, 1, 0, p0;\n\t"
        "selp.u32 t, 2, 0, p1;\n\tor.b32 %0, %0, t;\n\t}"
        : "=&r"(m) : "r"(a), "r"(parity_a), "r"(b), "r"(parity_b) : "memory");
    return m;
}
// Bounded wait: returns false when the phase did not complete within the budget (the caller records a status
// code and carries on; nothing spins forever).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t max_polls = 1u << 22) {
    for (uint32_t i = 0; i < max_polls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 64) __nanosleep(32);
    }
    return false;
}

// After a wait has given up, peers may still be sending into this CTA's shared memory (messages it stopped waiting
// for).  A CTA must not leave the cluster under them, so the error path idles for longer than a peer's own bounded
// waits can last before it tears down.  Bounded; reached only with an error status already recorded.
__device__ __forceinline__ void linger_after_timeout() {
    for (uint32_t i = 0; i < (1u << 21); ++i) __nanosleep(256);
}

// ---------------------------------------------------------------- tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t ncols) {      // one full warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {         // the allocating warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 lanes x 32 columns of fp32: thread i of the warp receives lane (base lane + i), columns [col, col+32)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 32 lanes x 8 columns of fp32 (for loops that are kept rolled to save instruction space)
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&v)[8]) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ---------------------------------------------------------------- MMA descriptors
// Shared-memory matrix descriptor, 128-byte swizzle: start address and the two byte offsets in 16-byte units,
// descriptor version 1 (bit 46), layout type SWIZZLE_128B = 2 (bits 61..63).  Tiles are 1024-byte aligned.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// The 14-bit start-address field of a matrix descriptor.  A shared::cta address taken inside a cluster can carry
// the CTA rank in its upper bits, so the field is masked, never added into the descriptor.
__device__ __forceinline__ uint64_t desc_addr(uint32_t addr) { return (uint64_t)((addr >> 4) & 0x3FFF); }
// Instruction descriptor for kind::f16 with bf16 operands and fp32 accumulation.
__host__ __device__ constexpr uint32_t idesc_bf16_f32(int M, int N, bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]; issued by one thread
__device__ __forceinline__ void mma_bf16_ss(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    uint32_t acc = accumulate ? 1u : 0u;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// One lane of a converged warp (the one that issues the products while the whole warp runs the control flow)
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
// arrive on an mbarrier of this CTA when all MMAs issued so far by this thread have completed
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

}  // namespace sm100
