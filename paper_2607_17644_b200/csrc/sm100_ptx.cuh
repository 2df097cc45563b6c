// Device-side building blocks for sm_100a: mbarrier (with bounded waits), TMA tiled loads,
// tcgen05 tensor-core MMA with TMEM accumulators, and the operand descriptors they consume.
// Header-only; every function is a thin wrapper over one PTX instruction or one descriptor word.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace laga {

// ------------------------------------------------------------------------------------------------
// Status word (one per launch, in caller-provided workspace).  A kernel that gives up on a wait
// records why and where, then unwinds normally: nothing traps and nothing spins forever.
// ------------------------------------------------------------------------------------------------
constexpr unsigned int kStatusOk = 0u;
constexpr unsigned int kStatusTimeout = 0x54000000u;   // | site id in the low bits
constexpr unsigned int kStatusCheck = 0x43000000u;     // a device-side self-check failed; | site id

// Wall-clock budget of a single mbarrier wait.  Kernels here run for milliseconds; a wait that has
// not completed after this long means a protocol bug, and the kernel unwinds instead of hanging.
constexpr unsigned long long kWaitBudgetNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

// ------------------------------------------------------------------------------------------------
// mbarrier
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

// Shared by every role of a CTA: once set, all later waits return at once so the CTA can unwind.
struct AbortFlag {
    volatile uint32_t value;
};

// Bounded wait.  Returns true when the phase completed; false after the budget ran out or another
// role already aborted (the status word then names the first site that gave up).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, AbortFlag* abort_flag,
                                          unsigned int* status, uint32_t site,
                                          unsigned long long budget_ns = kWaitBudgetNs) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    uint32_t polls = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++polls & 0xffu) == 0u) {
            if (abort_flag->value != 0u) return false;
            if (global_timer_ns() - t0 > budget_ns) {
                abort_flag->value = 1u;
                if (status) atomicCAS(status, kStatusOk, kStatusTimeout | site);
                return false;
            }
        }
    }
}

// Warp-uniform variant for code that goes on to execute warp-collective (.sync.aligned)
// instructions: every lane gets the same answer.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, AbortFlag* abort_flag,
                                               unsigned int* status, uint32_t site,
                                               unsigned long long budget_ns = kWaitBudgetNs) {
    // (every lane polls: one polling lane plus a warp broadcast measured 10-17 % slower kernels)
    const bool ok = mbar_wait(bar, parity, abort_flag, status, site, budget_ns);
    return __all_sync(0xffffffffu, ok);
}

// ------------------------------------------------------------------------------------------------
// Checked build.  Compiled with -DLAGA_DEBUG, every TMA issue and every global store of the kernels first
// verifies its own index arithmetic (coordinate alignment, row / column bounds, pointer alignment).  A
// failed check records kStatusCheck | site in the status word and the access is SKIPPED: the kernel runs
// on (a skipped load shows up as a bounded-wait timeout at worst), nothing traps, and the host reads
// LAGA_ERR_DEVICE_CHECK with the site from laga_query_status.  In the normal build the checks vanish.
// ------------------------------------------------------------------------------------------------
#ifdef LAGA_DEBUG
constexpr bool kDeviceChecks = true;
#else
constexpr bool kDeviceChecks = false;
#endif
__device__ __forceinline__ bool device_check(bool cond, unsigned int* status, uint32_t site) {
    if (!kDeviceChecks || cond) return true;
    if (status) atomicCAS(status, kStatusOk, kStatusCheck | (site & 0xffffffu));
    return false;
}
__device__ __forceinline__ bool aligned16_dev(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0u; }

// ------------------------------------------------------------------------------------------------
// Unwinding after a wait gave up.  A role that leaves its loop early may still have asynchronous work in
// flight that targets this CTA's shared memory or TMEM: TMA copies it armed, MMAs it issued.  Before the CTA
// frees TMEM and exits, the producer lane waits (1 ms at most per barrier, whatever the abort flag says) for
// the copies it armed, and the MMA lane commits to a barrier of its own and waits for that.
// ------------------------------------------------------------------------------------------------
constexpr unsigned long long kQuiesceBudgetNs = 1000000ull;
__device__ __forceinline__ void mbar_wait_quiesce(uint64_t* bar, uint32_t parity) {
    const unsigned long long t0 = global_timer_ns();
    while (!mbar_try_wait(bar, parity))
        if (global_timer_ns() - t0 > kQuiesceBudgetNs) return;
}
// The barriers a producer lane has armed with expect_tx, with the parity of the phase each was last armed
// for: two bit masks over the CTA's barrier array (all barriers of a kernel sit in one array of fewer than
// 64), so the record lives in registers.
struct ArmedBarriers {
    uint64_t* base;
    uint64_t armed = 0ull, parity = 0ull;
    __device__ __forceinline__ explicit ArmedBarriers(uint64_t* barrier_array) : base(barrier_array) {}
    __device__ __forceinline__ void arm(uint64_t* b, uint32_t ph) {
        const uint64_t bit = 1ull << static_cast<uint32_t>(b - base);
        armed |= bit;
        parity = (ph & 1u) ? (parity | bit) : (parity & ~bit);
    }
    __device__ __forceinline__ void quiesce() const {
        for (uint32_t i = 0; i < 64u; ++i)
            if ((armed >> i) & 1ull) mbar_wait_quiesce(base + i, static_cast<uint32_t>((parity >> i) & 1ull));
    }
};

// ------------------------------------------------------------------------------------------------
// Programmatic dependent launch.  A kernel launched with the programmatic-stream-serialization attribute may
// start while the kernel before it in the stream is still running: its CTAs take SMs as they free up and run
// their set-up (barrier init, TMEM allocation, descriptor prefetch), then every thread waits here until the
// preceding grid has completed and its memory is visible.  NOTHING global may be read or written before the
// wait.  Every kernel of the library executes both calls, so completion is transitive along a chain of
// launches; without the launch attribute they return at once.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ------------------------------------------------------------------------------------------------
// TMA (tiled bulk tensor copies global -> shared, completion on an mbarrier)
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
// x is the innermost (contiguous) coordinate; x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, uint64_t* bar, int x,
                                            int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}

// TMA store of one box from shared memory (bulk async-group completion).  The shared-memory source must have
// been written, fenced into the async proxy (fence_async_shared) and the writers synchronised before the issue.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, const void* smem_src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Wait until at most `kPending` of this thread's store groups still READ their shared-memory source.
template <int kPending>
__device__ __forceinline__ void tma_store_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kPending) : "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// The same with the checked build's self-check: x on a 16-byte boundary (the hardware raises an illegal
// instruction otherwise), y not negative, destination slab 1024-byte aligned.
__device__ __forceinline__ void tma_load_2d_chk(unsigned int* status, void* smem_dst, const CUtensorMap* map, uint64_t* bar,
                                                int x, int y) {
    if (device_check((x & 7) == 0 && x >= 0 && y >= 0 && (smem_u32(smem_dst) & 1023u) == 0u, status, 0xE00000u | (x & 0xffff)))
        tma_load_2d(smem_dst, map, bar, x, y);
}

// ------------------------------------------------------------------------------------------------
// TMEM allocation (one warp executes these, all 32 lanes converged)
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t n_cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(smem_result)),
                 "r"(n_cols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t n_cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(n_cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// ------------------------------------------------------------------------------------------------
// Operand descriptors
// ------------------------------------------------------------------------------------------------
// Shared-memory matrix descriptor for a 128-byte-swizzled operand tile.  The tile is a stack of
// "slabs"; a slab is R rows of 128 bytes (64 bf16), rows 8 apart are 1024 bytes apart, and the 16-byte
// chunk index within a row is XORed with (row & 7) -- exactly what a TMA box of 64 bf16 x R rows with
// CU_TENSOR_MAP_SWIZZLE_128B writes when the slab base is 1024-byte aligned.
//   K-major operand (rows = M or N index, the 64 contiguous elements run along K):
//       stride byte offset  = 1024 (next group of 8 rows); leading byte offset unused.
//       One MMA consumes K = 16 elements = 32 bytes: advance the start address by 32 bytes per K step
//       inside a slab, and by the slab size every 64 elements of K.
//   MN-major operand (rows = K index, the 64 contiguous elements run along M or N):
//       stride byte offset  = 1024 (next group of 8 K rows)
//       leading byte offset = slab size (next 64 elements along M/N).
//       One MMA consumes 16 K rows: advance the start address by 2048 bytes per K step.
constexpr uint64_t kDescSwizzle128B = 2ull << 61;
constexpr uint64_t kDescVersionSm100 = 1ull << 46;

__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr, uint32_t leading_bytes,
                                                   uint32_t stride_bytes) {
    return static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4) |
           (static_cast<uint64_t>((leading_bytes & 0x3ffffu) >> 4) << 16) |
           (static_cast<uint64_t>((stride_bytes & 0x3ffffu) >> 4) << 32) | kDescVersionSm100 | kDescSwizzle128B;
}
__device__ __forceinline__ uint64_t desc_k_major(uint32_t smem_addr) {
    return make_smem_desc(smem_addr, 16u, 1024u);
}
__device__ __forceinline__ uint64_t desc_mn_major(uint32_t smem_addr, uint32_t slab_bytes) {
    return make_smem_desc(smem_addr, slab_bytes, 1024u);
}

// Instruction descriptor for kind::f16 with bf16 inputs and fp32 accumulation.
// a_mn_major / b_mn_major: 0 = K-major operand, 1 = MN-major operand.
__host__ __device__ constexpr uint32_t make_idesc_bf16(int m, int n, int a_mn_major, int b_mn_major) {
    return (1u << 4)                                   // D format  : fp32
           | (1u << 7)                                 // A format  : bf16
           | (1u << 10)                                // B format  : bf16
           | (static_cast<uint32_t>(a_mn_major) << 15)
           | (static_cast<uint32_t>(b_mn_major) << 16)
           | (static_cast<uint32_t>(n >> 3) << 17)
           | (static_cast<uint32_t>(m >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------
// tcgen05 MMA / commit / TMEM load-store.  MMA and commit are issued by ONE thread.
// ------------------------------------------------------------------------------------------------
// D[tmem] (+)= A[smem] * B[smem]; accumulate == 0 overwrites D.
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]; A holds packed bf16 pairs, one 32-bit column per two K elements.
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Chains of MMAs from ONE asm block.  The issuing lane shares its scheduler with two busy softmax warps and runs at
// four to six clocks per instruction, so the ten or so instructions that the compiler spends on every separately
// written MMA (descriptor arithmetic in 64 bits, predicate set-up, operand moves) are time the tensor pipe
// idles: measured, the lane's instruction count sets the tile period once it exceeds the MMAs' own time.  Here a
// step costs two additions and the MMA: the descriptor's upper word is constant and its lower word (start
// address in 16-byte units, below the leading-offset field) is advanced by an immediate.
#define LAGA_MMA_TS_STEP(AOFF, BOFF, P)                                                       \
    "add.u32 a, %1, " #AOFF ";\n\tadd.u32 lo, %2, " #BOFF ";\n\tmov.b64 desc, {lo, %3};\n\t"  \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], desc, %4, " #P ";\n\t"
// Each chain comes in two parts, so that the lane can put the bookkeeping that follows a chain BEFORE the
// chain's last MMAs: it then runs while the pipe still has those queued (the queue holds only two to four MMAs).
#define LAGA_MMA_COMMIT2(B0, B1)                                                                               \
    "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [" #B0 "];\n\t"                      \
    "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [" #B1 "];\n\t"
// S = Q K^T for one 96-key tile: twelve K steps, A = Q from TMEM (8 columns per step), B = a K-major key tile of
// three slabs of 96 rows (12288 bytes = 768 descriptor units each; 32 bytes = 2 units per step inside a slab).
// Head: the steps of slabs 0 and 1 (the first overwrites S).  Tail: slab 2, then commits to two mbarriers
// (shared-memory addresses).
__device__ __forceinline__ void mma_ts_chain_qk96_head(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b32 a, lo;\n\t.reg .b64 desc;\n\t"
        "setp.ne.b32 p0, 0, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
        LAGA_MMA_TS_STEP(0, 0, p0) LAGA_MMA_TS_STEP(8, 2, p1) LAGA_MMA_TS_STEP(16, 4, p1) LAGA_MMA_TS_STEP(24, 6, p1)
        LAGA_MMA_TS_STEP(32, 768, p1) LAGA_MMA_TS_STEP(40, 770, p1) LAGA_MMA_TS_STEP(48, 772, p1) LAGA_MMA_TS_STEP(56, 774, p1)
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc)
        : "memory");
}
__device__ __forceinline__ void mma_ts_chain_qk96_tail(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                                       uint32_t bar0, uint32_t bar1) {
    asm volatile(
        "{\n\t.reg .pred p1;\n\t.reg .b32 a, lo;\n\t.reg .b64 desc;\n\t"
        "setp.eq.b32 p1, 0, 0;\n\t"
        LAGA_MMA_TS_STEP(64, 1536, p1) LAGA_MMA_TS_STEP(72, 1538, p1) LAGA_MMA_TS_STEP(80, 1540, p1) LAGA_MMA_TS_STEP(88, 1542, p1)
        LAGA_MMA_COMMIT2(%5, %6)
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(bar0), "r"(bar1)
        : "memory");
}
// O (+)= P V for one 96-key tile: six K steps, A = P from TMEM (8 columns per step), B = an MN-major value tile
// (16 key rows = 2048 bytes = 128 descriptor units per step).  Head: three steps, accumulate_first == 0
// overwrites O.  Tail: three steps, then commits to two mbarriers.
__device__ __forceinline__ void mma_ts_chain_pv96_head(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                                       uint32_t accumulate_first) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b32 a, lo;\n\t.reg .b64 desc;\n\t"
        "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
        LAGA_MMA_TS_STEP(0, 0, p0) LAGA_MMA_TS_STEP(8, 128, p1) LAGA_MMA_TS_STEP(16, 256, p1)
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate_first)
        : "memory");
}
__device__ __forceinline__ void mma_ts_chain_pv96_tail(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                                       uint32_t bar0, uint32_t bar1) {
    asm volatile(
        "{\n\t.reg .pred p1;\n\t.reg .b32 a, lo;\n\t.reg .b64 desc;\n\t"
        "setp.eq.b32 p1, 0, 0;\n\t"
        LAGA_MMA_TS_STEP(24, 384, p1) LAGA_MMA_TS_STEP(32, 512, p1) LAGA_MMA_TS_STEP(40, 640, p1)
        LAGA_MMA_COMMIT2(%5, %6)
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(bar0), "r"(bar1)
        : "memory");
}

// The chains of the backward kernels (128-row slabs: 16384 bytes = 1024 descriptor units per 64 elements of K).
#define LAGA_MMA_SS_STEP(OFF, P)                                                                                  \
    "add.u32 lo, %1, " #OFF ";\n\tmov.b64 da, {lo, %2};\n\tadd.u32 lo, %3, " #OFF ";\n\tmov.b64 db, {lo, %4};\n\t"  \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, " #P ";\n\t"
#define LAGA_MMA_COMMIT1(B0) "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [" #B0 "];\n\t"
// D = A B^T, both operands K-major tiles of 128 rows in shared memory, 192 deep (twelve steps); then one commit.
__device__ __forceinline__ void mma_ss_chain12_k128(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                                    uint32_t idesc, uint32_t bar0) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b32 lo;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p0, 0, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
        LAGA_MMA_SS_STEP(0, p0) LAGA_MMA_SS_STEP(2, p1) LAGA_MMA_SS_STEP(4, p1) LAGA_MMA_SS_STEP(6, p1)
        LAGA_MMA_SS_STEP(1024, p1) LAGA_MMA_SS_STEP(1026, p1) LAGA_MMA_SS_STEP(1028, p1) LAGA_MMA_SS_STEP(1030, p1)
        LAGA_MMA_SS_STEP(2048, p1) LAGA_MMA_SS_STEP(2050, p1) LAGA_MMA_SS_STEP(2052, p1) LAGA_MMA_SS_STEP(2054, p1)
        LAGA_MMA_COMMIT1(%6)
        "}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(bar0)
        : "memory");
}
// The same, 128 deep (eight steps).
__device__ __forceinline__ void mma_ss_chain8_k128(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                                   uint32_t idesc, uint32_t bar0) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b32 lo;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p0, 0, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
        LAGA_MMA_SS_STEP(0, p0) LAGA_MMA_SS_STEP(2, p1) LAGA_MMA_SS_STEP(4, p1) LAGA_MMA_SS_STEP(6, p1)
        LAGA_MMA_SS_STEP(1024, p1) LAGA_MMA_SS_STEP(1026, p1) LAGA_MMA_SS_STEP(1028, p1) LAGA_MMA_SS_STEP(1030, p1)
        LAGA_MMA_COMMIT1(%6)
        "}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(bar0)
        : "memory");
}
// D (+)= A B: A = packed bf16 in TMEM (8 columns per step), B = an MN-major tile of 128 rows of K (16 rows = 2048
// bytes = 128 units per step), eight steps; accumulate_first == 0 overwrites D; then two commits.
__device__ __forceinline__ void mma_ts_chain8_mn(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                                 uint32_t accumulate_first, uint32_t bar0, uint32_t bar1) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b32 a, lo;\n\t.reg .b64 desc;\n\t"
        "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
        LAGA_MMA_TS_STEP(0, 0, p0) LAGA_MMA_TS_STEP(8, 128, p1) LAGA_MMA_TS_STEP(16, 256, p1) LAGA_MMA_TS_STEP(24, 384, p1)
        LAGA_MMA_TS_STEP(32, 512, p1) LAGA_MMA_TS_STEP(40, 640, p1) LAGA_MMA_TS_STEP(48, 768, p1) LAGA_MMA_TS_STEP(56, 896, p1)
        LAGA_MMA_COMMIT2(%6, %7)
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate_first), "r"(bar0), "r"(bar1)
        : "memory");
}
// The same with A in two blocks of 32 columns that lie 64 columns apart (the dQ kernel's dS); then one commit.
__device__ __forceinline__ void mma_ts_chain8_mn_split(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                                       uint32_t accumulate_first, uint32_t bar0) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b32 a, lo;\n\t.reg .b64 desc;\n\t"
        "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
        LAGA_MMA_TS_STEP(0, 0, p0) LAGA_MMA_TS_STEP(8, 128, p1) LAGA_MMA_TS_STEP(16, 256, p1) LAGA_MMA_TS_STEP(24, 384, p1)
        LAGA_MMA_TS_STEP(64, 512, p1) LAGA_MMA_TS_STEP(72, 640, p1) LAGA_MMA_TS_STEP(80, 768, p1) LAGA_MMA_TS_STEP(88, 896, p1)
        LAGA_MMA_COMMIT1(%6)
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate_first), "r"(bar0)
        : "memory");
}
// D = A B^T: A = packed bf16 in TMEM (8 columns per step), B = a K-major tile of 128 rows, 128 deep (eight steps);
// overwrites D; then two commits.
__device__ __forceinline__ void mma_ts_chain8_k128(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                                   uint32_t bar0, uint32_t bar1) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b32 a, lo;\n\t.reg .b64 desc;\n\t"
        "setp.ne.b32 p0, 0, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
        LAGA_MMA_TS_STEP(0, 0, p0) LAGA_MMA_TS_STEP(8, 2, p1) LAGA_MMA_TS_STEP(16, 4, p1) LAGA_MMA_TS_STEP(24, 6, p1)
        LAGA_MMA_TS_STEP(32, 1024, p1) LAGA_MMA_TS_STEP(40, 1026, p1) LAGA_MMA_TS_STEP(48, 1028, p1) LAGA_MMA_TS_STEP(56, 1030, p1)
        LAGA_MMA_COMMIT2(%5, %6)
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(bar0), "r"(bar1)
        : "memory");
}
__device__ __forceinline__ uint32_t desc_lo(uint64_t desc) { return static_cast<uint32_t>(desc); }
__device__ __forceinline__ uint32_t desc_hi(uint64_t desc) { return static_cast<uint32_t>(desc >> 32); }

// Arrive (count 1) on `bar` once every MMA this thread issued so far has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                     smem_u32(bar))
                 : "memory");
}

// Shared memory -> TMEM, issued by ONE thread like an MMA (and executed in order with that thread's MMAs): row r
// of a 128-row K-major swizzled slab, bytes [0, 32) from the descriptor's start address, lands in TMEM lane r,
// columns [col, col + 8) -- the layout in which an MMA reads sixteen bf16 of its A operand from TMEM.  Advance
// the start address by 32 bytes per eight columns inside a slab, exactly as for an MMA's K steps.  Completion is
// observed through mma_commit.
__device__ __forceinline__ void tmem_cp_128x256b(uint32_t taddr, uint64_t desc) {
    asm volatile("tcgen05.cp.cta_group::1.128x256b [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}

// Warp-collective TMEM loads.  Lane l of warp w (w % 4 selects the 32-lane quarter) receives, from
// TMEM lane 32*(w%4)+l, the 32-bit columns [col, col+N).  `taddr` = (lane << 16) | column.
__device__ __forceinline__ void tmem_ld_x32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
          "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
          "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
          "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st_x32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_x16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st_wait() {
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// ------------------------------------------------------------------------------------------------
// CTA pairs (cluster of two, tcgen05 cta_group::2)
// ------------------------------------------------------------------------------------------------
// One thread of the even CTA issues an MMA that runs on both SMs: D has 256 rows (rows 0..127 in the even
// CTA's TMEM, 128..255 in the odd CTA's, at the same column address), each CTA supplies its own 128 rows of
// A and HALF of the N columns of B from its own shared memory, at the same offsets in both CTAs.  What the
// pair saves is shared-memory traffic: every CTA fills and reads half a B tile instead of a whole one.
__device__ __forceinline__ uint32_t cluster_cta_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address, in the cluster-wide shared window, of the object at `local` in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t cluster_map(const void* local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(local)), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load into THIS CTA's shared memory whose bytes are counted on a barrier given by its cluster address
// (the even CTA's barrier: its MMA thread waits for both halves).  Each CTA fetches its own half itself.
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(x), "r"(y)
        : "memory");
}
// ---- distributed shared memory between the two CTAs of a cluster (used by the fused backward) ----------
// 16-byte store into the peer's shared memory (generic proxy), at a cluster address from cluster_map().
__device__ __forceinline__ void st_shared_cluster_v4(uint32_t cluster_addr, uint4 v) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
// Orders this thread's generic-proxy writes (local or peer shared memory) before later async-proxy reads
// (tcgen05.mma operand fetches) of the same data: issue after the stores, before signalling the consumer.
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
// try_wait that acquires at cluster scope: the waiter goes on to read data the PEER CTA wrote.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, AbortFlag* abort_flag, unsigned int* status,
                                                  uint32_t site, unsigned long long budget_ns = kWaitBudgetNs) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    uint32_t polls = 0;
    while (true) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((++polls & 0xffu) == 0u) {
            if (abort_flag->value != 0u) return false;
            if (global_timer_ns() - t0 > budget_ns) {
                abort_flag->value = 1u;
                if (status) atomicCAS(status, kStatusOk, kStatusTimeout | site);
                return false;
            }
        }
    }
}
// tcgen05.commit (one-CTA MMAs) that arrives on the barrier at this offset in every CTA of `cta_mask`: how the
// MMA lane of one CTA tells its PEER that the MMAs which read a buffer have completed.  Signals only; no data.
__device__ __forceinline__ void mma_commit_to(uint64_t* bar, uint16_t cta_mask) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(cta_mask)
                 : "memory");
}
// fp32 reduction into global memory without a return value (one lane, one element; a warp whose lanes hit 32
// consecutive floats makes one 128-byte transaction).
__device__ __forceinline__ void red_add_f32(float* addr, float v) {
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(addr), "f"(v) : "memory");
}

__device__ __forceinline__ void tma_load_2d_pair_chk(unsigned int* status, void* smem_dst, const CUtensorMap* map,
                                                     uint32_t bar_cluster_addr, int x, int y) {
    if (device_check((x & 7) == 0 && x >= 0 && y >= 0 && (smem_u32(smem_dst) & 1023u) == 0u, status, 0xE00000u | (x & 0xffff)))
        tma_load_2d_pair(smem_dst, map, bar_cluster_addr, x, y);
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t n_cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(n_cols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t n_cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(n_cols) : "memory");
}
__device__ __forceinline__ void mma_ss_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// Arrive (count 1) on the barrier at this offset in every CTA of `cta_mask` once the pair's MMAs issued so far
// have completed.
__device__ __forceinline__ void mma_commit_pair(uint64_t* bar, uint16_t cta_mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(cta_mask)
                 : "memory");
}

// ------------------------------------------------------------------------------------------------
// Small helpers
// ------------------------------------------------------------------------------------------------
// 256-bit global accesses (sm_100): a lane moves 32 contiguous bytes per instruction.  The row-per-lane epilogues
// and operand stagings of the attention kernels touch 32 different lines per instruction whatever its width, so
// halving the instruction count halves what they cost the load/store unit.  The address must be 32-byte aligned.
__device__ __forceinline__ void st_global_v8(void* addr, const uint32_t* r) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]),
                 "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void ld_global_v8(const void* addr, uint32_t* r) {
    asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "l"(addr));
}
__device__ __forceinline__ bool aligned32_dev(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0u; }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);   // .x = lo (low 16 bits), .y = hi
    return *reinterpret_cast<uint32_t*>(&v);
}

}  // namespace laga
