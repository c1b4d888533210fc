// Thin wrappers over the sm_100a instructions the tensor-core kernels use: mbarrier, TMA tiled
// loads (no multicast), tcgen05 (tensor memory allocation, UMMA, commit, TMEM loads), and the
// shared-memory / instruction descriptors.  Every wait is bounded: after about a second it
// records where it gave up in a status word and the kernel winds down instead of spinning.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace dlf {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Optional timeline probe (compiled in only with -DDLF_TRACE): CTA 0 stores the global timer at
// a few points after the status word.
#ifdef DLF_TRACE
#define DLF_TRACE_POINT(status, slot) do { if (blockIdx.x == 0) reinterpret_cast<volatile unsigned long long*>(status)[4 + (slot)] = global_ns(); } while (0)
// per-phase cycle sums of CTA 0's thread 0: ACC adds the cycles since the last mark to a slot
#define DLF_TRACE_DECL(acc, mark) long long acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}; long long mark = clock64()
#define DLF_TRACE_ACC(acc, slot, mark) do { const long long now_ = clock64(); acc[slot] += now_ - mark; mark = now_; } while (0)
#define DLF_TRACE_FLUSH(status, acc) do { if (blockIdx.x == 0 && threadIdx.x == 0) for (int i_ = 0; i_ < 8; i_++) reinterpret_cast<volatile long long*>(status)[4 + i_] = acc[i_]; } while (0)
// the same for any one thread of CTA 0, into slots base .. base + 7
#define DLF_TRACE_FLUSH_AT(status, acc, base) do { if (blockIdx.x == 0) for (int i_ = 0; i_ < 8; i_++) reinterpret_cast<volatile long long*>(status)[4 + (base) + i_] = acc[i_]; } while (0)
// ... the first n accounts only (the status block holds 28 slots)
#define DLF_TRACE_FLUSH_N(status, acc, base, n) do { if (blockIdx.x == 0) for (int i_ = 0; i_ < (n); i_++) reinterpret_cast<volatile long long*>(status)[4 + (base) + i_] = acc[i_]; } while (0)
#else
#define DLF_TRACE_POINT(status, slot) do { } while (0)
#define DLF_TRACE_DECL(acc, mark) do { } while (0)
#define DLF_TRACE_ACC(acc, slot, mark) do { } while (0)
#define DLF_TRACE_FLUSH(status, acc) do { } while (0)
#define DLF_TRACE_FLUSH_AT(status, acc, base) do { } while (0)
#define DLF_TRACE_FLUSH_N(status, acc, base, n) do { } while (0)
#endif

// ---- programmatic dependent launch -----------------------------------------------------------------
// A kernel launched with the programmatic-serialization attribute may start while its predecessor
// in the stream still runs: its CTAs are scheduled as SMs free up and run their set-up (barriers,
// TMEM allocation, bias staging); pdl_wait() then blocks until the predecessor grid has completed
// and its memory operations are visible.  Both are no-ops for a normal launch.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- mbarrier ---------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_inval(uint64_t* bar) {
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
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

constexpr uint64_t kWaitLimitNs = 1000000000ull;  // one second

// Waits for the phase with the given parity.  `abort_flag` is a CTA-shared word: once any wait
// of the CTA has given up, every later wait returns at once so that all roles drain.  On
// giving up, `code` (which wait, which CTA) is stored in the global status word.  HOT marks the waits on
// the critical path between two layers of a fused group: they keep polling much longer before they
// start to sleep.  (try_wait with a suspend-time hint instead of this loop was measured 1-3 % slower.)
// The polling loop is a function of its own (one copy per kernel instead of one per wait site: a kernel has dozens of
// waits, and their inlined loops made up a large part of its code); the first poll, which usually succeeds, stays inline.
template <bool HOT>
__device__ __noinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status, int code,
                                            uint64_t limit_ns) {
    uint64_t t0 = 0;   // the global timer is read only once a wait has lasted a while
    uint32_t spins = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        // back off: a spinning single-thread role shares its scheduler with the warps doing the work
        if (spins > (HOT ? 2048u : 4u)) __nanosleep(spins > 64 && !HOT ? 128 : 32);
        if ((++spins & 63u) == 0) {
            if (*abort_flag) return false;
            const uint64_t now = global_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > limit_ns) {
                *abort_flag = 1;
                atomicCAS(status, 0, code);
                return false;
            }
        }
    }
}
template <bool HOT = false>
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          int* status, int code, uint64_t limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow<HOT>(bar, parity, abort_flag, status, code, limit_ns);
}

// Warp-wide form: every lane polls (a whole warp stays on the issue path so that the addresses it
// computes are warp-uniform values); the result is voted so that the warp leaves a wait together.
template <bool HOT = false>
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                               int* status, int code) {
    const bool ok = mbar_wait<HOT>(bar, parity, abort_flag, status, code);
    return __all_sync(0xffffffffu, ok);
}

// True in exactly one lane of a converged warp (the same lane every time).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .b32 rx;\n\t.reg .pred px;\n\t"
        "elect.sync rx|px, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, px;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// Makes generic-proxy writes to shared memory visible to the async proxy (TMA, UMMA operand reads).
__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---- TMA (tiled mode, one CTA, no multicast) ------------------------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1,
                                            int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1,
                                            int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3)
        : "memory");
}

__device__ __forceinline__ void tma_load_5d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1,
                                            int c2, int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3), "r"(c4)
        : "memory");
}

// ---- tcgen05: tensor memory ---------------------------------------------------------------------
// Allocation is warp-wide; the base address is written to shared memory.
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// Shared-memory matrix descriptor, K-major operand, 128-byte swizzle: rows of 64 fp16 (128 bytes),
// eight rows per 1024-byte swizzle atom, atoms of consecutive row groups 1024 bytes apart.
// The swizzle is a function of the absolute shared-memory address (bits 7..9 select the XOR of
// bits 4..6), so a start address on any 128-byte row of a 1024-byte-aligned buffer is valid with
// base-offset field left at zero.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= static_cast<uint64_t>(1) << 16;                        // leading byte offset (unused here)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;                // stride byte offset between row groups
    d |= static_cast<uint64_t>(1) << 46;                        // descriptor version of this architecture
    d |= static_cast<uint64_t>(2) << 61;                        // 128-byte swizzle
    return d;
}
// Instruction descriptor: fp16 x fp16 -> fp32, both operands K-major, M = 128, given N.
__host__ __device__ constexpr uint32_t umma_idesc_f16(int n) {
    return (1u << 4) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(128 >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]; issued by one thread.
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                         uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Measured on B200 (M = 128, K = 16, fp16): an issue loop run by ONE thread (`if (lane == 0)`) spends
// about 72 cycles per UMMA whatever N is, because every descriptor is a per-thread value that has to
// be moved into uniform registers; the same loop run by the whole warp with warp-uniform descriptors
// and the UMMA group under elect_one() reaches the hardware's rates: 48 cycles at N = 64 (operand
// reads from shared memory), N / 2 cycles from N = 128 up.  Descriptors differ only in the 14-bit
// start-address field, so stepping one is a 64-bit add of (bytes >> 4).
//
// Lean 32-bit form (older issue loops): the descriptors' upper words are constants, only the
// start-address field of the lower word changes from one MMA to the next.
constexpr uint32_t kDescHiSw128 = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t saddr) { return ((saddr & 0x3FFFFu) >> 4) | (1u << 16); }
__device__ __forceinline__ void umma_f16_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %6};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHiSw128)
        : "memory");
}

// The four K = 16 steps of one 64-channel chunk in a single statement: A and B advance by 32 bytes (2 units) per step, both
// descriptors share the constant high word.  The first step accumulates only if `accumulate` is non-zero.
__device__ __forceinline__ void umma_f16_x4(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t.reg .b32 ta, tb;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "mov.b64 da, {%1, %5};\n\tmov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
        "setp.eq.b32 p, %3, %3;\n\t"
        "add.u32 ta, %1, 2;\n\tadd.u32 tb, %2, 2;\n\tmov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
        "add.u32 ta, %1, 4;\n\tadd.u32 tb, %2, 4;\n\tmov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
        "add.u32 ta, %1, 6;\n\tadd.u32 tb, %2, 6;\n\tmov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHiSw128)
        : "memory");
}

// ---- TMA store (shared -> global, tiled, clipped at the tensor's edges) ---------------------------
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* m, const void* src, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until the committed stores have finished READING shared memory (the buffer may be reused).
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... all but the newest committed store have finished reading.
__device__ __forceinline__ void tma_store_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
// ... all but the newest `pending` (0..3) committed stores of this thread have finished reading.
__device__ __forceinline__ void tma_store_wait_read_n(int pending) {
    if (pending <= 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    else if (pending == 1) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
    else if (pending == 2) asm volatile("cp.async.bulk.wait_group.read 2;" ::: "memory");
    else asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// The barrier gets one arrival when every UMMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// 32 lanes x 16 consecutive fp32 columns: thread t of the warp gets lane (taddr.lane + t).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; i++) v[i] = __uint_as_float(r[i]);
}

// Two 16-column loads in flight before one wait: 32 consecutive fp32 columns of the thread's lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; i++) v[i] = __uint_as_float(r[i]);
}

// Split form: the load is issued into raw registers and waited for later, so that the next chunk's
// load is in flight while this chunk is being worked on.  The wait names the registers as in/out
// operands: nothing that reads them can be scheduled ahead of it.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld32_wait(uint32_t (&r)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31]) : : "memory");
}

template <int ACT>
__device__ __forceinline__ float act_t(float v) {
    if (ACT >= 1) v = fmaxf(v, 0.0f);
    if (ACT == 2) v = fminf(v, 6.0f);
    return v;
}

__device__ __forceinline__ float apply_act(float v, int act) {
    if (act >= 1) v = fmaxf(v, 0.0f);
    if (act == 2) v = fminf(v, 6.0f);
    return v;
}

__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
// Two values rounded to fp16, then clamped to [lo, hi] as a pair.  Rounding is monotone and the bounds used (0, 6, the
// infinities) are fp16 values, so clamping after the rounding gives the same bits as clamping before it - at one
// instruction per bound and PAIR instead of one per bound and value.
__device__ __forceinline__ uint32_t pack_half2_clamp(float a, float b, __half2 lo, __half2 hi) {
    const __half2 h = __hmin2(__hmax2(__floats2half2_rn(a, b), lo), hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}
// The activation of a rounded pair: none, ReLU, ReLU6.
template <int ACT>
__device__ __forceinline__ __half2 act_h2(__half2 h) {
    if (ACT >= 1) h = __hmax2(h, __float2half2_rn(0.0f));
    if (ACT == 2) h = __hmin2(h, __float2half2_rn(6.0f));
    return h;
}

}  // namespace dlf
