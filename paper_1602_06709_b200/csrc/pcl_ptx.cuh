// Thin inline-PTX wrappers for sm_100a: mbarrier, TMA (cp.async.bulk.tensor),
// tcgen05 (TMEM allocation, UMMA issue/commit, TMEM loads) and the bounded
// wait used by every pipeline in this library.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace pcl {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ----------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// (warp-collective, like the copies it arms: the whole producer warp executes it and one elected lane arrives)
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t"
                 "@pe mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t}" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Every wait in this library goes through here.  It polls the barrier until it
// completes, for at most the wait limit of wall time (checked every 64 polls), and
// gives up at once if another role of the CTA has already given up.  On expiry
// it records `code` in the device status word (0 = fine; read and cleared by
// pcl_last_device_status()), raises the CTA's abort flag and returns false;
// callers then leave their loops and fall through to the common teardown, so the
// kernel always terminates.
// The limit lives next to the status word (status_word[1], in microseconds; 2 s unless a test shortens it): it is
// read only on the slow path, when a wait has already polled 64 times without success.
constexpr unsigned int kDefaultWaitMicros = 2000000u;      // 2 s; real waits last micro- to milliseconds
__device__ __forceinline__ unsigned long long wait_limit_nanos(const unsigned int* status_word) {
    return 1000ull * *reinterpret_cast<const volatile unsigned int*>(status_word + 1);
}

__device__ __forceinline__ unsigned long long global_nanos() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ bool bounded_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                             unsigned int* status_word, uint32_t code) {
    unsigned long long t0 = 0, limit = 0;
    for (uint32_t spin = 0;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 63u) {
            if (*abort_flag) return false;
            const unsigned long long now = global_nanos();
            if (t0 == 0) { t0 = now; limit = wait_limit_nanos(status_word); }
            else if (now - t0 > limit) break;
            __nanosleep(64);
        }
    }
    *abort_flag = 1u;
    atomicCAS(status_word, 0u, code);
    return false;
}

// Warp-uniform form: every lane polls, and the warp proceeds only if all lanes
// saw the barrier complete (keeps .sync.aligned instructions convergent even on
// the give-up path).
__device__ __forceinline__ bool bounded_wait_warp(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                  unsigned int* status_word, uint32_t code) {
    const bool ok = bounded_wait(bar, parity, abort_flag, status_word, code);
    return __all_sync(0xffffffffu, ok);
}

// Low-duty form for warps that wait long (an epilogue warp waits for a whole main loop): lane 0 polls and
// sleeps between polls, so that the wait takes almost no issue slots from the pipeline roles' loops
// that share the warp scheduler; the result is broadcast.
__device__ __forceinline__ bool bounded_wait_warp_relaxed(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                          unsigned int* status_word, uint32_t code) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) {
        unsigned long long t0 = 0, limit = 0;
        ok = 0;
        for (uint32_t spin = 0;; ++spin) {
            if (mbar_try_wait(bar, parity)) { ok = 1; break; }
            __nanosleep(200);
            if ((spin & 15u) == 15u) {
                if (*abort_flag) break;
                const unsigned long long now = global_nanos();
                if (t0 == 0) { t0 = now; limit = wait_limit_nanos(status_word); }
                else if (now - t0 > limit) {
                    *abort_flag = 1u;
                    atomicCAS(status_word, 0u, code);
                    break;
                }
            }
        }
    }
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// Explicit shared-memory vector accesses (32-bit shared address): the staging tile of the epilogue is reached through
// a pointer whose address space the compiler cannot see, and generic accesses would be ordered against the global
// stores around them.
__device__ __forceinline__ void st_shared_v4(uint32_t addr, float x, float y, float z, float w) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}
__device__ __forceinline__ float4 ld_shared_v4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

// ---------------------------------------------------------------------- TMA
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* m) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1, int c2,
                                            int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_load_5d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1, int c2,
                                            int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3), "r"(c4)
        : "memory");
}

// ---- TMA stores (shared -> global) in bulk async-groups
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* m, uint32_t src, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all earlier groups of this thread have finished READING their shared-memory source
__device__ __forceinline__ void bulk_wait_group_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... have completed
__device__ __forceinline__ void bulk_wait_group0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// makes shared-memory writes of this thread visible to the async proxy (TMA)
__device__ __forceinline__ void fence_proxy_async_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ------------------------------------------------------------------ tcgen05
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], TF32 operands, fp32 accumulate.
// Warp-collective (like every MMA, commit and k-step form below): the WHOLE warp executes it, converged, with the same
// operands in every lane, and one elected lane issues the instruction.  A loop that runs in lane 0 alone is divergent
// code to the compiler, which then moves every descriptor into the uniform registers the instruction takes, one word at
// a time; measured on a loop of nothing but MMAs: 54.5 cycles per MMA issued from lane 0 alone, 24.9 from a converged
// warp with an elected lane.
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p, pe;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Makes `bar` complete one arrival once all previously issued UMMAs of this thread are done.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t"
                 "@pe tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(smem_u32(bar))
                 : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread t of the warp gets lane (base_lane + t).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
// fp32 -> TF32 (10-bit mantissa), round to nearest even: what a TMA load through a TFLOAT32 tensor map does to
// an operand.  For operand tiles that threads write to shared memory themselves.
__device__ __forceinline__ float to_tf32(float x) {
    uint32_t r;
    asm("cvt.rn.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}
// Barrier among `count` threads (a multiple of 32) of the CTA; id 1-15 (0 is __syncthreads()).
__device__ __forceinline__ void named_barrier_sync(uint32_t id, uint32_t count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
// Zero 32 lanes x 32 consecutive fp32 columns (the counterpart of tmem_ld_32x32).
__device__ __forceinline__ void tmem_st_32x32_zero(uint32_t taddr) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, "
        "%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};"
        ::"r"(taddr), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ------------------------------------------------------- CTA pairs (cta_group::2)
// Two CTAs of a cluster (ranks 2i, 2i+1) run one M = 256 MMA: each holds its own 128 rows of A and half
// of the B rows at the same shared-memory offsets, the even CTA (the leader) issues.  Loads of either
// CTA may complete on the leader's barrier; a commit can arrive on the same barrier of both CTAs.
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
__device__ __forceinline__ uint32_t nclusters_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
    return r;
}
// shared::cluster address of `p` (a shared-memory object of this CTA) in the CTA of rank `rank`
__device__ __forceinline__ uint32_t map_to_cta(const void* p, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(void* dst, const CUtensorMap* m, uint32_t bar_cluster_addr, int c0,
                                                 int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(void* dst, const CUtensorMap* m, uint32_t bar_cluster_addr, int c0,
                                                 int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_load_5d_pair(void* dst, const CUtensorMap* m, uint32_t bar_cluster_addr, int c0,
                                                 int c1, int c2, int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3), "r"(c4)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_tf32_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p, pe;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// One arrival on `bar` (same offset) in both CTAs of the pair once the issued pair MMAs are done.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
    asm volatile("{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t"
                 "@pe tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
                 ::"r"(smem_u32(bar)), "h"(static_cast<uint16_t>(3))
                 : "memory");
}

// ------------------------------------------------- lean forms for the pipeline roles' loops
// The producer and the MMA-issuing role are each one warp that executes a chain of dependent instructions (all lanes
// the same values, one elected lane issuing), so every instruction costs several cycles of the k-step budget (a
// 128 x 256 x 32 k-step is 512 tensor cycles; measured: a loop of ~100 instructions per k-step held the tensor pipe at
// 63 %).  These forms take shared-memory addresses as 32-bit registers that the loops advance by addition, and issue the
// four K = 8 MMAs of a k-step from one asm block.
__device__ __forceinline__ bool mbar_try_wait_addr(uint32_t bar_addr, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar_addr), "r"(parity)
        : "memory");
    return ok != 0;
}
static __device__ __noinline__ bool bounded_wait_slow(uint32_t bar_addr, uint32_t parity, volatile uint32_t* abort_flag,
                                               unsigned int* status_word, uint32_t code) {
    unsigned long long t0 = 0, limit = 0;
    for (uint32_t spin = 0;; ++spin) {
        if (mbar_try_wait_addr(bar_addr, parity)) return true;
        if ((spin & 63u) == 63u) {
            if (*abort_flag) return false;
            const unsigned long long now = global_nanos();
            if (t0 == 0) { t0 = now; limit = wait_limit_nanos(status_word); }
            else if (now - t0 > limit) break;
            __nanosleep(64);
        }
    }
    *abort_flag = 1u;
    atomicCAS(status_word, 0u, code);
    return false;
}
// One poll inline (the common case); the bounded polling loop is out of line.
__device__ __forceinline__ bool bounded_wait_addr(uint32_t bar_addr, uint32_t parity, volatile uint32_t* abort_flag,
                                                  unsigned int* status_word, uint32_t code) {
    if (mbar_try_wait_addr(bar_addr, parity)) return true;
    return bounded_wait_slow(bar_addr, parity, abort_flag, status_word, code);
}
// True in the lane that elect.sync picks for a full, converged warp (the same lane every time for the same mask, so it
// is the lane that issues in the elected-lane forms).
__device__ __forceinline__ bool elected_lane() {
    uint32_t e;
    asm volatile("{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\tselp.u32 %0, 1, 0, pe;\n\t}" : "=r"(e));
    return e != 0;
}
// Warp-collective wait: every lane polls; the warp goes on only if all lanes saw the barrier complete, so that the
// lanes stay together (the elected-lane forms below need a converged warp) on the give-up path too.
__device__ __forceinline__ bool bounded_wait_addr_warp(uint32_t bar_addr, uint32_t parity, volatile uint32_t* abort_flag,
                                                       unsigned int* status_word, uint32_t code) {
    const bool ok = bounded_wait_addr(bar_addr, parity, abort_flag, status_word, code);
    return __all_sync(0xffffffffu, ok);
}
__device__ __forceinline__ void mbar_expect_tx_addr(uint32_t bar_addr, uint32_t bytes) {
    asm volatile("{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t"
                 "@pe mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t}" ::"r"(bar_addr), "r"(bytes) : "memory");
}
template <bool kPair>
__device__ __forceinline__ void umma_commit_addr(uint32_t bar_addr) {
    if constexpr (kPair)
        asm volatile("{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t"
                     "@pe tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
                     ::"r"(bar_addr), "h"(static_cast<uint16_t>(3))
                     : "memory");
    else
        asm volatile("{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t"
                     "@pe tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar_addr)
                     : "memory");
}
// Warp-collective (the whole producer warp executes them, one elected lane issues the copy).
// TMA loads with 32-bit shared addresses; kPair: the barrier is a shared::cluster address (the leader's).
template <bool kPair>
__device__ __forceinline__ void tma_load_3d_addr(uint32_t dst, const CUtensorMap* m, uint32_t bar, int c0, int c1, int c2) {
    if constexpr (kPair)
        asm volatile(
            "{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t@pe cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];\n\t}"
            ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t@pe cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];\n\t}"
            ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
template <bool kPair>
__device__ __forceinline__ void tma_load_4d_addr(uint32_t dst, const CUtensorMap* m, uint32_t bar, int c0, int c1, int c2,
                                                 int c3) {
    if constexpr (kPair)
        asm volatile(
            "{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t@pe cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];\n\t}"
            ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t@pe cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];\n\t}"
            ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
template <bool kPair>
__device__ __forceinline__ void tma_load_5d_addr(uint32_t dst, const CUtensorMap* m, uint32_t bar, int c0, int c1, int c2,
                                                 int c3, int c4) {
    if constexpr (kPair)
        asm volatile(
            "{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t@pe cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];\n\t}"
            ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t@pe cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];\n\t}"
            ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
// The four K = 8 MMAs of one k-step (32 reduction elements).  Descriptors are given as their low words (the
// address field lives there) plus the constant high words; k-block kk is kAStep / kBStep sixteen-byte units
// further (2 for a K-major 128-byte row, 64 for an MN-major tile whose 8-deep reduction groups are 1 KB apart).
// `acc_first` = 0 makes the first MMA overwrite the accumulator.
#define PCL_UMMA_KSTEP_BODY(CG)                                                                                   \
    asm volatile(                                                                                                 \
        "{\n\t.reg .pred p, pe;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"                                    \
        "setp.ne.b32 p, %6, 0;\n\t"                                                                               \
        "elect.sync _|pe, 0xffffffff;\n\t"                                                                        \
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %4};\n\t"                                                      \
        "@pe tcgen05.mma.cta_group::" CG ".kind::tf32 [%0], da, db, %5, p;\n\t"                                    \
        "setp.ne.b32 p, 1, 0;\n\t"                                                                                \
        "add.u32 al, %1, %7;\n\tadd.u32 bl, %2, %8;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %4};\n\t"          \
        "@pe tcgen05.mma.cta_group::" CG ".kind::tf32 [%0], da, db, %5, p;\n\t"                                    \
        "add.u32 al, al, %7;\n\tadd.u32 bl, bl, %8;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %4};\n\t"          \
        "@pe tcgen05.mma.cta_group::" CG ".kind::tf32 [%0], da, db, %5, p;\n\t"                                    \
        "add.u32 al, al, %7;\n\tadd.u32 bl, bl, %8;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %4};\n\t"          \
        "@pe tcgen05.mma.cta_group::" CG ".kind::tf32 [%0], da, db, %5, p;\n\t}"                                   \
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(a_hi), "r"(b_hi), "r"(idesc), "r"(acc_first), "n"(kAStep),       \
        "n"(kBStep)                                                                                               \
        : "memory")
template <bool kPair, int kAStep, int kBStep>
__device__ __forceinline__ void umma_kstep_tf32(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t a_hi,
                                                uint32_t b_hi, uint32_t idesc, uint32_t acc_first) {
    if constexpr (kPair) PCL_UMMA_KSTEP_BODY("2");
    else PCL_UMMA_KSTEP_BODY("1");
}
#undef PCL_UMMA_KSTEP_BODY
// The same with a K-major A (k-block = 2 units) and the k-block stride of B in a register (2: K-major, 64: MN-major).
// `nsl` (1..4): how many of the four K = 8 slices are issued; the rest are known to multiply zeros only (few-channel
// layers pack fewer than 32 live reduction elements into a block) and are skipped by a guard predicate.
#define PCL_UMMA_KSTEP_BODY_BS(CG)                                                                                \
    asm volatile(                                                                                                 \
        "{\n\t.reg .pred p, pe, q2, q3, q4;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"                        \
        "setp.ne.b32 p, %6, 0;\n\t"                                                                               \
        "elect.sync _|pe, 0xffffffff;\n\t"                                                                        \
        "setp.gt.u32 q2, %8, 1;\n\tsetp.gt.u32 q3, %8, 2;\n\tsetp.gt.u32 q4, %8, 3;\n\t"                          \
        "and.pred q2, q2, pe;\n\tand.pred q3, q3, pe;\n\tand.pred q4, q4, pe;\n\t"                                \
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %4};\n\t"                                                      \
        "@pe tcgen05.mma.cta_group::" CG ".kind::tf32 [%0], da, db, %5, p;\n\t"                                    \
        "setp.ne.b32 p, 1, 0;\n\t"                                                                                \
        "add.u32 al, %1, 2;\n\tadd.u32 bl, %2, %7;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %4};\n\t"           \
        "@q2 tcgen05.mma.cta_group::" CG ".kind::tf32 [%0], da, db, %5, p;\n\t"                                    \
        "add.u32 al, al, 2;\n\tadd.u32 bl, bl, %7;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %4};\n\t"           \
        "@q3 tcgen05.mma.cta_group::" CG ".kind::tf32 [%0], da, db, %5, p;\n\t"                                    \
        "add.u32 al, al, 2;\n\tadd.u32 bl, bl, %7;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %4};\n\t"           \
        "@q4 tcgen05.mma.cta_group::" CG ".kind::tf32 [%0], da, db, %5, p;\n\t}"                                   \
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(a_hi), "r"(b_hi), "r"(idesc), "r"(acc_first), "r"(b_step),       \
        "r"(nsl)                                                                                                  \
        : "memory")
template <bool kPair>
__device__ __forceinline__ void umma_kstep_tf32_bs(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t a_hi,
                                                   uint32_t b_hi, uint32_t idesc, uint32_t acc_first, uint32_t b_step,
                                                   uint32_t nsl) {
    if constexpr (kPair) PCL_UMMA_KSTEP_BODY_BS("2");
    else PCL_UMMA_KSTEP_BODY_BS("1");
}
#undef PCL_UMMA_KSTEP_BODY_BS

// Shared-memory matrix descriptor (64-bit) for a swizzled operand tile.
//   bits  0-13 start address >> 4      bits 16-29 leading byte offset >> 4
//   bits 32-45 stride byte offset >> 4 bits 46-47 descriptor version (1 on sm_100)
//   bits 61-63 swizzle mode: 2 = 128-byte rows swizzled in 16-byte chunks,
//                            1 = 128-byte rows swizzled in 32-byte chunks
// K-major tile (mode 2; rows of 128 B = 32 fp32 along the reduction): 8-row groups
// are `sbo` bytes apart, the leading offset is unused.
// MN-major tile of 32-bit elements (mode 1 is the only one the hardware takes for
// tf32; rows of 128 B = 32 fp32 along M or N, one row per reduction index, the
// swizzle pattern repeats every 4 rows): 32-element column groups are `lbo` bytes
// apart, 4-row reduction groups are `sbo` bytes apart.
constexpr uint32_t kSwizzle128B = 2, kSwizzle128B_Atom32B = 1;
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes,
                                                   uint32_t swizzle_mode) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;
    d |= static_cast<uint64_t>(swizzle_mode) << 61;
    return d;
}

// Instruction descriptor for kind::tf32, fp32 accumulator, M = 128 (256 for a CTA pair).
//   bits 4-5 D format (1 = f32)   bits 7-9 A format (2 = tf32)   bits 10-12 B format
//   bit 15 A is MN-major          bit 16 B is MN-major
//   bits 17-22 N >> 3             bits 24-28 M >> 4
__host__ __device__ constexpr uint32_t make_idesc_tf32(uint32_t n, bool a_mn_major, bool b_mn_major,
                                                       uint32_t m = 128u) {
    return (1u << 4) | (2u << 7) | (2u << 10) | (static_cast<uint32_t>(a_mn_major) << 15) |
           (static_cast<uint32_t>(b_mn_major) << 16) | ((n >> 3) << 17) | ((m >> 4) << 24);
}

// Wait codes recorded in the device status word (which role gave up).
enum : uint32_t {
    WAIT_PRODUCER_EMPTY = 0x101,
    WAIT_MMA_FULL = 0x102,
    WAIT_MMA_TMEM_EMPTY = 0x103,
    WAIT_EPI_TMEM_FULL = 0x104,
    WAIT_DRAIN = 0x105,
    WAIT_ISSUE_TURN = 0x106,
};

}  // namespace pcl
