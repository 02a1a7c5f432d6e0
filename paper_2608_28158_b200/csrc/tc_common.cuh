// sm_100a building blocks shared by the tensor-core kernels: mbarrier (bounded waits), TMA tile
// loads/stores, tcgen05 MMA / TMEM access, UMMA shared-memory and instruction descriptors.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace harts {
namespace tc {

// A wait that ran out reports this code in the status word and latches a flag shared by the CTA: every later
// wait of that CTA returns at once, its loops end, tensor memory is released (results are garbage, nothing hangs).
constexpr int STATUS_TIMEOUT = 1;
constexpr unsigned long long WAIT_LIMIT_NS = 500ull * 1000 * 1000;   // wall time per wait; a healthy wait takes microseconds

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier ------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  `dead` points to the CTA's latch in shared memory (0 at kernel start).  Returns false when the wait
// gave up: because this one ran out of time (the latch and the status word are then set), or because the latch was
// already set by an earlier one.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* status, volatile int* dead,
                                          unsigned long long limit_ns = WAIT_LIMIT_NS) {
    if (*dead) return false;
    // a healthy wait ends within these polls; the timer is consulted only after them
#pragma unroll 1
    for (int i = 0; i < 2048; i++) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 255) == 255 && *dead) return false;
    }
    const unsigned long long t0 = global_ns();
    for (int round = 0; round < (1 << 24); round++) {            // the poll count is bounded too, should the timer stall
#pragma unroll 1
        for (int i = 0; i < 32; i++)
            if (mbar_try(bar, parity)) return true;
        if (*dead) return false;
        if (global_ns() - t0 > limit_ns) break;
    }
    *dead = 1;
    if (status) atomicExch(status, STATUS_TIMEOUT);
    return false;
}
// The same for a whole (converged) warp: one lane polls, so that 31 lanes do not spend shared-memory cycles on it.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, int* status, volatile int* dead) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, status, dead);
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
// Last wait of a CTA that is giving up: waits (bounded, whatever the latch says) for a copy or MMA group still in
// flight, so that nothing lands in shared or tensor memory after the CTA has gone.
__device__ __forceinline__ void mbar_wait_drain(uint64_t* bar, uint32_t parity) {
    const unsigned long long t0 = global_ns();
    for (int round = 0; round < (1 << 20); round++) {
        if (mbar_try(bar, parity)) return;
        if (global_ns() - t0 > 20ull * 1000 * 1000) return;
    }
}
// Fixed pause (about 0.2 ms, bounded) of a CTA that is giving up and cannot name the barriers of its loads in flight.
__device__ __forceinline__ void drain_delay() {
    const unsigned long long t0 = global_ns();
    for (int i = 0; i < (1 << 20) && global_ns() - t0 < 200000ull; i++) {}
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

// Adds expected bytes to the barrier's current phase without arriving (for a phase whose copies are requested in
// several instalments; the last instalment arrives with mbar_expect_tx).
__device__ __forceinline__ void mbar_expect_tx_only(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

// ---- flags between CTAs of one launch --------------------------------------------------------------------------------------
// A CTA that has produced something another CTA of the same launch consumes publishes a flag in global memory; the
// consumer polls it.  Every writer of the data fences before the CTA-wide barrier that precedes flag_set; the consumer
// reads the data only after flag_wait returned true and a CTA-wide barrier.  The wait is bounded like the others (a
// longer limit: the producer may be a long sequence), honours the CTA's latch, and ends as soon as the launch's status
// word shows that some CTA has given up, so that one time-out does not become a chain of them.
constexpr unsigned long long FLAG_WAIT_LIMIT_NS = 4000ull * 1000 * 1000;
__device__ __forceinline__ void flag_set(int* flag) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(flag), "r"(1) : "memory");
}
__device__ __forceinline__ bool flag_wait(const int* flag, int* status, volatile int* dead,
                                          unsigned long long limit_ns = FLAG_WAIT_LIMIT_NS) {
    const unsigned long long t0 = global_ns();
    for (int round = 0; round < (1 << 26); round++) {
        int v;
#pragma unroll 1
        for (int i = 0; i < 16; i++) {
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
            if (v != 0) return true;
        }
        if (*dead) return false;
        // another CTA of the launch has already given up (its wait ran out): what this one waits for may never come
        if (status && *reinterpret_cast<volatile int*>(status) != 0) {
            *dead = 1;
            return false;
        }
        if (global_ns() - t0 > limit_ns) break;
    }
    *dead = 1;
    if (status) atomicExch(status, STATUS_TIMEOUT);
    return false;
}

// ---- fences ---------------------------------------------------------------------------------------
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---- TMA (tile mode, no multicast) -------------------------------------------------------------------
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, const void* smem_src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(map), "r"(smem_u32(smem_src)), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ---- tensor memory ---------------------------------------------------------------------------------
template <int COLS>
__device__ __forceinline__ void tmem_alloc(uint32_t* slot_in_smem) {   // one full warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot_in_smem)),
                 "r"(COLS));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
}
template <int COLS>
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr) {         // the same warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(COLS));
}

// 32 lanes x 32 columns of 32-bit: thread i of the warp gets columns [col, col+32) of lane (lane_base + i)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,"
        "%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}
// 16 lanes x 16 columns of 32-bit in the layout of a matrix fragment: with c = lane & 3, m = lane >> 2 thread `lane`
// gets r[0..1] = lane m, columns 2c, 2c+1; r[2..3] = lane m + 8, same columns; r[4..7] = the same for columns + 8.
// The address's lane field selects which 16 lanes (base or base + 16 of the warp's quarter).
__device__ __forceinline__ void tmem_ld_frag16(uint32_t taddr, uint32_t* r) {
    asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
}
// Four 8x8 matrices of 16-bit elements between fragments and shared memory, transposed on the way: thread 8m + r
// gives the address of the 16-byte row r of matrix m; a fragment register holds two consecutive elements of what is a
// column of the matrix in memory.
__device__ __forceinline__ void stmatrix_x4_trans(uint32_t saddr, const uint32_t* r) {
    asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1,%2,%3,%4};"
                 ::"r"(saddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t saddr, uint32_t* r) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(saddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,"
        "%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---- UMMA descriptors (bf16 operands in 128-byte-swizzled panels of [rows][64 elements]) -----------------
// Shared-memory matrix descriptor: start address, leading and stride byte offsets (each >> 4),
// descriptor version 1, layout type 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor for kind::f16 with bf16 inputs and fp32 accumulation.
// major: 0 = the operand's K dimension is contiguous in shared memory, 1 = its M/N dimension is.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int a_major, int b_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_major << 15) | ((uint32_t)b_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// The same with the A operand in tensor memory: lane = row m, two bf16 per 32-bit column, a k-step of 16 covers 8 columns.
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// Byte offset of element (r, c) inside a 128-byte-swizzled panel of [rows][64 bf16].
__device__ __forceinline__ uint32_t sw128(int r, int c) {
    return r * 128 + ((((c * 2) >> 4) ^ (r & 7)) << 4) + ((c * 2) & 15);
}
// Byte offset of the 16-byte chunk `ch` (0..7) of row r.
__device__ __forceinline__ uint32_t sw128_chunk(int r, int ch) { return r * 128 + ((ch ^ (r & 7)) << 4); }

// Operand descriptor for a tile whose K dimension is contiguous: panels of [ROWS][64] over K, k-step ks
// covers 16 elements.
template <int ROWS>
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t tile, int ks) {
    return smem_desc(tile + (ks >> 2) * (ROWS * 128) + (ks & 3) * 32, 16, 1024);
}
// Operand descriptor for a tile stored [K rows][M/N columns] (M/N contiguous): panels of [KROWS][64] over
// M/N, k-step ks covers 16 rows.
template <int KROWS>
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t tile, int ks) {
    return smem_desc(tile + ks * 2048, KROWS * 128, 1024);
}

// The same descriptors split into a loop-invariant base (k-step 0) and a k-step increment of the start-address
// field, so that the issuing thread only adds a constant per MMA.
__device__ __forceinline__ uint64_t desc_kmajor_base(uint32_t tile) { return smem_desc(tile, 16, 1024); }
template <int ROWS>
__host__ __device__ constexpr uint64_t kstep_kmajor(int ks) {
    return (uint64_t)(((ks >> 2) * (ROWS * 128) + (ks & 3) * 32) >> 4);
}
template <int KROWS>
__device__ __forceinline__ uint64_t desc_mnmajor_base(uint32_t tile) { return smem_desc(tile, KROWS * 128, 1024); }
__host__ __device__ constexpr uint64_t kstep_mnmajor(int ks) { return (uint64_t)((ks * 2048) >> 4); }

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

}  // namespace tc
}  // namespace harts
