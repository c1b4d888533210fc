// Single-layer implicit-GEMM convolution on the tcgen05 tensor cores (general stride; the
// kernel of every group that holds one dense convolution the fused-chain kernel does not take).
//
//   D[m, n] = sum over (tap, ci) of A_tap[m, ci] * W[n, tap, ci]        (Eq. 1 counts these MACs)
//   M = 128 output pixels (a TN x TH x TW patch), N = up to 256 output channels, K = taps x C_in.
//
// A persistent grid of `sm_count` CTAs (the SM-count knob) walks the (pixel tile, channel tile)
// work list.  Per CTA: four producer threads (measured on B200: one TMA instruction keeps its
// issuing thread busy for about 0.28 us whatever the box size, so the loads of a stage are spread
// over several warps) issue TMA tiled loads (the tap's shifted, strided
// window of the NHWC input, zero-filled outside the image = the convolution's padding; and the
// tap's [C_out][64] weight slab) into a ring of 128-byte-swizzled stages; one thread issues
// tcgen05.mma (fp16 x fp16 -> fp32) into one of two TMEM accumulators; sixteen epilogue warps (four
// per TMEM lane quarter, interleaved 32-column chunks: with two per quarter the schedulers sat idle on
// the dependent load / add / pack / store chains, measured 1.8 us per 128 x 256 tile) drain the other
// accumulator: bias (staged
// in shared memory), residual, activation, fp16 rounding.  Without pooling the tile is written to
// a swizzled staging buffer (two of them where the ring leaves room) and a separate warp sends it
// off with TMA stores (clipped at the tensor's edges), waits until they have read the buffer and hands
// it back - so the epilogue warps never wait for a store.  A residual is fetched by that same warp
// with TMA loads straight INTO the staging buffer one or two tiles ahead and added in place: with one
// output pixel per thread, direct residual loads would touch 32 cache lines per instruction and
// were measured to double the time of the memory-bound 1x1 layers.  With the fused 2x2 max-pool
// the window is reduced by warp shuffles and written with 16-byte stores.
// Row mode (3x3, stride 1, whole 64-channel chunks, images up to 126 pixels wide): a tile is whole output rows seen
// with a pitch of W + 2, so the three taps of a kernel row are ONE loaded window read through UMMA descriptors that
// start 0, 1 and 2 pixels into it; the window crosses L2 -> shared memory three times per chunk instead of nine.
// Chosen where it cuts the bytes a CTA streams by a fifth or more (measured: 64 -> 128 at 112x112 34 -> 23 us,
// 512 -> 512 at 14x14 23 -> 17 us, the ResNet-50 3x3 layers 8 % faster; neutral where the weight slabs dominate).
// The epilogue is specialised at compile time on (activation, pool, residual): it is the part of
// the kernel that bounds memory-bound layers, and runtime branches there cost more than the math.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstdio>
#include <cstring>

#include "internal.h"
#include "ptx.cuh"

namespace dlf {

namespace {

constexpr int kEpiParts = 4;                // epilogue warps per TMEM lane quarter; each takes every kEpiParts-th 32-column chunk
constexpr int kEpiWarps = 4 * kEpiParts;
constexpr int kMmaWarp = kEpiWarps;         // warps 0..15 epilogue (warp & 3 = TMEM lane quarter), then the UMMA issuer,
constexpr int kProdWarp0 = kEpiWarps + 1;   // four producers: A even / A odd / B even / B odd ring stages,
constexpr int kMaxOutBufs = 4;               // staging buffers of finished tiles
constexpr int kStoreWarp = kProdWarp0 + 4;  // and one warp for the TMA stores of finished tiles and the TMA loads of residual tiles
constexpr int kThreads = 32 * (kEpiWarps + 6);
constexpr int kABytes = 128 * 128;  // 128 pixels x 64 fp16
constexpr int kMaxSmem = 232448 - 1024;  // dynamic part: the 227 KB per-CTA limit minus the static barriers
constexpr size_t kSplitCounterBytes = 65536;  // head of the split-K workspace: arrival counters, then the partial tiles

struct ConvTcParams {
    int N, Ho, Wo, Cout;
    int kh, kw, stride, pad;
    int TW, TH, TN, rows, tiles_w, tiles_h, tiles_n;  // rows = TW * TH * TN <= 128 pixels of a tile
    int BN, n_tiles_n, acc_stride;
    int kchunks, ksteps_last;
    int a_bytes;               // one 64-channel slab of the tile's pixels in a ring stage: rows rounded up to 8, x 128 bytes
    int tps, tgroups;          // taps per ring stage (3 = a whole kernel row, see the row mode) and tap groups per K-chunk group
    int kg, kgroups, grouped;  // K chunks per ring stage; stages per tap; 1 = 5-d / 4-d maps (cin % 64 == 0)
    int stages;
    int store_depth;              // TMA stores of finished tiles in flight (1 .. out_bufs)
    int n_work;
    int stage_out_off, bias_off;  // byte offsets in dynamic shared memory
    int out_bufs, out_buf_bytes;  // staging buffers (1 or 2) and the size of one
    int splits, kgs;              // split-K: work items per tile and K-chunk groups per item (1 / kgroups without)
    float* partial;               // split-K: fp32 partial tiles [tile][split][row][acc_stride]
    int* counters;                // split-K: arrivals per (tile, epilogue warp); zero between launches
    uint32_t tmem_cols;
    int kchunks1, stride2;        // second source: 64-channel chunks kchunks1 .. kchunks-1 of K come from it, read with stride2
    const float* bias;
    const float* bias2;           // second source's bias (added to the first's), or null
    const __half* res;
    __half* out;
    int* status;
};

struct TileCoord {
    int n0, ho0, wo0, co0;
    int tile, ks;  // split-K: the tile's number and which share of K this work item takes
};

template <bool SPLIT = false>
__device__ __forceinline__ TileCoord decode_work(const ConvTcParams& p, int t) {
    TileCoord c;
    c.ks = 0;
    if (SPLIT) {   // the shares of one tile are neighbours in the work list: they run side by side
        c.ks = t % p.splits;
        t /= p.splits;
    }
    c.tile = t;
    const int nt = t % p.n_tiles_n;
    int mt = t / p.n_tiles_n;
    c.co0 = nt * p.BN;
    c.wo0 = (mt % p.tiles_w) * p.TW;
    mt /= p.tiles_w;
    c.ho0 = (mt % p.tiles_h) * p.TH;
    c.n0 = (mt / p.tiles_h) * p.TN;
    return c;
}

// Device-wide barrier of a multi-layer launch (all CTAs resident, one per SM): every CTA adds one to a counter in global
// memory when it has finished a layer; a warp that is about to read what another CTA wrote in an earlier layer of the same
// launch first waits until the counter has reached `target` = layers finished x CTAs.  Bounded like every other wait.
struct GridSync {
    unsigned* counter;   // null: a single-layer launch, nothing to wait for
    unsigned target;
};
__device__ __forceinline__ bool grid_wait(const GridSync& gs, int lane, volatile int* abort_flag, int* status) {
    if (gs.counter == nullptr || gs.target == 0u) return true;
    bool ok = true;
    if (lane == 0) {
        uint64_t t0 = 0;
        uint32_t spins = 0;
        while (true) {
            unsigned v;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(gs.counter) : "memory");
            if (v >= gs.target) break;
            if (spins > 8) __nanosleep(64);
            if ((++spins & 63u) == 0) {
                if (*abort_flag) { ok = false; break; }
                const uint64_t now = global_ns();
                if (t0 == 0) t0 = now;
                if (now - t0 > kWaitLimitNs) {
                    *abort_flag = 1;
                    atomicCAS(status, 0, 0x700 | (blockIdx.x << 12));
                    ok = false;
                    break;
                }
            }
        }
        __threadfence();
        if (gs.target == gridDim.x && threadIdx.x == 32 * kProdWarp0) DLF_TRACE_POINT(status, 27);
    }
    ok = __all_sync(0xffffffffu, ok);
    // what the other CTAs stored (TMA stores) is read here through the async proxy (TMA loads) as well
    asm volatile("fence.proxy.async;" ::: "memory");
    return ok;
}

// The barriers of one CTA (static shared memory of the kernel that calls the roles).
struct ConvBars {
    uint64_t *full_bar, *empty_bar, *tfull_bar, *tempty_bar, *sfull_bar, *sfree_bar;
    int* abort_s;
};

// The warp roles of one layer: everything between the CTA's set-up (barriers initialised, tensor memory allocated) and
// its wind-down.  Called once by the single-layer kernel and once per layer by the multi-layer kernel.
template <int ACT, bool POOL, bool RES, bool ROW, bool SPLIT>
__device__ __forceinline__ void conv_tc_roles(const CUtensorMap* tmx_p, const CUtensorMap* tmw_p, const CUtensorMap* tmy_p,
                                              const CUtensorMap* tmr_p, const CUtensorMap* tmx2_p, const CUtensorMap* tmw2_p,
                                              const ConvTcParams& p, const ConvBars& sm, uint32_t tmem_base,
                                              uint8_t* stage0, uint32_t base, const GridSync& gs) {
    float* bias_s = reinterpret_cast<float*>(stage0 + p.bias_off);
    constexpr int kTps = ROW ? 3 : 1;   // taps per ring stage: a whole kernel row in the row mode
    const int stage_bytes = p.kg * (p.a_bytes + kTps * p.BN * 128);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = sm.abort_s;
    const int k_iters = p.tgroups * p.kgroups;

    if (warp == kStoreWarp) {
        // ---- staging buffers out (TMA stores) and residual tiles in (TMA loads) ------------------------
        // One lane per 64-channel plane: a thread's bulk copies run one after the other (about 0.3 us each,
        // measured), the copies of different lanes side by side.
        if (!POOL && !SPLIT) {   // (split-K tiles leave through the partial sums in global memory)
            if (RES && !grid_wait(gs, lane, abort_flag, p.status)) return;   // the residual may be a layer of this launch
            uint8_t* stage_out = stage0 + p.stage_out_off;
            auto planes_of = [&](const TileCoord& c) { return (min(p.BN, ((p.Cout - c.co0) + 15) & ~15) + 63) >> 6; };
            auto fetch_residual = [&](int t, uint32_t b) {
                const TileCoord c = decode_work(p, t);
                const int planes = planes_of(c);
                if (lane == 0) mbar_expect_tx(&sm.sfree_bar[b], static_cast<uint32_t>(planes * p.rows) * 128u);
                __syncwarp();
                if (lane < planes)
                    tma_load_4d(stage_out + b * p.out_buf_bytes + lane * kABytes, tmr_p, &sm.sfree_bar[b], c.co0 + lane * 64, c.wo0, c.ho0, c.n0);
            };
            if (RES)
#pragma unroll 1
                for (int jj = 0; jj < p.out_bufs; jj++)
                    if (static_cast<int>(blockIdx.x) + jj * static_cast<int>(gridDim.x) < p.n_work) fetch_residual(blockIdx.x + jj * gridDim.x, jj);
            // Up to `store_depth` stores are in flight: a store takes about 1.5 us from its issue until it has read its
            // buffer whatever its size (measured), so a layer of short tiles (one or two loads each) that waited for
            // every store before the next was bound by that latency, not by any bandwidth.  Every lane commits a group
            // per tile (an empty one where it has no plane), so all lanes count the same groups.
            const int depth = p.store_depth, bufs = p.out_bufs;
            int b = 0, fb = 0;                // staging buffer of tile j / of the oldest store in flight
            uint32_t ph = 0;                  // phase of sfull[b]
            int t_free = blockIdx.x, j = 0;   // tile of the oldest store in flight
            DLF_TRACE_DECL(sacc, smark);  // cycles of CTA 0's store warp: 0 wait for a staged tile, 1 store and its read, 2 residual fetch
#pragma unroll 1
            for (int t = blockIdx.x; t < p.n_work; t += gridDim.x, j++) {
                if (!mbar_wait_warp(&sm.sfull_bar[b], ph, abort_flag, p.status, 0x500 | (blockIdx.x << 12))) break;
                DLF_TRACE_ACC(sacc, 0, smark);
                const TileCoord c = decode_work(p, t);
                if (lane < planes_of(c))
                    tma_store_4d(tmy_p, stage_out + b * p.out_buf_bytes + lane * kABytes, c.co0 + lane * 64, c.wo0, c.ho0, c.n0);
                tma_store_commit();
                if (++b == bufs) { b = 0; ph ^= 1u; }
                if (j + 1 >= depth) {
                    tma_store_wait_read_n(depth - 1);  // the oldest store has read its buffer: it may take the next residual / tile
                    __syncwarp();
                    DLF_TRACE_ACC(sacc, 1, smark);
                    const int t2 = t_free + bufs * static_cast<int>(gridDim.x);
                    if (RES) {
                        if (t2 < p.n_work) fetch_residual(t2, fb);
                    } else if (lane == 0) {
                        mbar_arrive(&sm.sfree_bar[fb]);
                    }
                    if (++fb == bufs) fb = 0;
                    t_free += gridDim.x;
                    DLF_TRACE_ACC(sacc, 2, smark);
                }
            }
            tma_store_wait_read();   // shared memory outlives every store that reads it
            __syncwarp();
            if (lane == 0) DLF_TRACE_FLUSH_N(p.status, sacc, 11, 3);
        }
    } else if (warp >= kProdWarp0) {
        // ---- producers: TMA loads into the stage ring -------------------------------------------
        // The warp stays converged; lane g loads the stage's g-th 64-channel chunk as a box of its own: the copies
        // of a stage run side by side (one thread's copies run one after the other) and every chunk starts on a
        // 1024-byte boundary whatever the tile's row count (a chunk that starts inside a swizzle atom costs the
        // tensor core twice the shared-memory reads).
        {
            const int role = warp - kProdWarp0;
            const bool is_b = role >= 2;
            // the first work item is decoded ahead of the wait for the previous kernel: the divisions (about a hundred
            // cycles each for a lone warp) then cost nothing on the path from that kernel's end to the first copy
            const TileCoord c_first = decode_work<SPLIT>(p, blockIdx.x);
            if (role == 0 && lane == 0 && gs.counter == nullptr) DLF_TRACE_POINT(p.status, 25);
            if (!is_b) {
                pdl_wait();
                if (!grid_wait(gs, lane, abort_flag, p.status)) return;   // the input may be a layer of this launch
            }
            const uint32_t parity = role & 1;
            const uint32_t my_bytes = static_cast<uint32_t>(p.kg) * (is_b ? static_cast<uint32_t>(kTps * p.BN) : static_cast<uint32_t>(p.rows)) * 128u;
            uint32_t it = 0;
            bool ok = true;
            DLF_TRACE_DECL(pacc, pmark);  // cycles of CTA 0's producers: 0 wait for a free stage, 1 issue
            // One ring stage: K-chunk group kq of tap group tg (row mode: tap group tg = kernel row tg, its window
            // loaded once at the row's first tap).  False once a wait has given up.
            // (ring position and phase are kept as counters: no division on the way to a copy)
            int ring_st = 0;
            uint32_t ring_ph = 0;
            auto load_stage = [&](const TileCoord& c, int tap, int r, int s, int kq) -> bool {
                const int st = ring_st;
                const uint32_t ph = ring_ph;
                if (++ring_st == p.stages) { ring_st = 0; ring_ph ^= 1u; }
                // a ring stage belongs to ONE producer warp of each kind: a warp that skipped a phase of
                // a stage's barrier could not tell "two phases ago" from "now" by parity
                if ((st & 1u) != parity) return true;
                if (!mbar_wait_warp(&sm.empty_bar[st], ph ^ 1u, abort_flag, p.status, 0x100 | (blockIdx.x << 12))) return false;
                DLF_TRACE_ACC(pacc, 0, pmark);
                if (it == 0 && role == 0 && lane == 0 && gs.counter == nullptr) DLF_TRACE_POINT(p.status, 26);
                uint8_t* sa = stage0 + static_cast<size_t>(st) * stage_bytes;
                if (lane == 0) mbar_expect_tx(&sm.full_bar[st], my_bytes);
                __syncwarp();
                if (lane < p.kg) {   // a chunk past C_in / 64 lies outside the tensor map and arrives as zeros
                    const int kc = kq * p.kg + lane;
                    const bool second = kc >= p.kchunks1;   // (1x1 layers with whole 64-channel chunks only: see conv_tc_dual_supported)
                    if (is_b) {
                        uint8_t* dst = sa + p.kg * p.a_bytes + lane * kTps * p.BN * 128;
                        if (second) tma_load_4d(dst, tmw2_p, &sm.full_bar[st], 0, c.co0, 0, kc - p.kchunks1);
                        else if (p.grouped) tma_load_4d(dst, tmw_p, &sm.full_bar[st], 0, c.co0, tap, kc);
                        else tma_load_3d(dst, tmw_p, &sm.full_bar[st], kc * 64, tap, c.co0);
                    } else {
                        const int wi = c.wo0 * p.stride - p.pad + s, hi = c.ho0 * p.stride - p.pad + r;
                        uint8_t* dst = sa + lane * p.a_bytes;
                        if (second) tma_load_5d(dst, tmx2_p, &sm.full_bar[st], 0, c.wo0 * p.stride2, c.ho0 * p.stride2, c.n0, kc - p.kchunks1);
                        else if (p.grouped) tma_load_5d(dst, tmx_p, &sm.full_bar[st], 0, wi, hi, c.n0, kc);
                        else tma_load_4d(dst, tmx_p, &sm.full_bar[st], kc * 64, wi, hi, c.n0);
                    }
                }
                __syncwarp();
                if (it == 0 && lane == 0) DLF_TRACE_POINT(p.status, 2);
                DLF_TRACE_ACC(pacc, 1, pmark);
                return true;
            };
#pragma unroll 1
            for (int t = blockIdx.x; t < p.n_work && ok; t += gridDim.x) {
                const TileCoord c = t == static_cast<int>(blockIdx.x) ? c_first : decode_work<SPLIT>(p, t);
                if (SPLIT) {   // this item's share of the tile's (tap group, K-chunk group) list
                    const int l0 = c.ks * p.kgs, l1 = min(k_iters, l0 + p.kgs);
#pragma unroll 1
                    for (int li = l0; li < l1 && ok; li++, it++) {
                        const int tg = li / p.kgroups, tap = tg * kTps;
                        ok = load_stage(c, tap, tap / p.kw, tap % p.kw, li - tg * p.kgroups);
                    }
                } else {
                    int r = 0, s = 0;   // kernel row and column of the tap group's first tap
#pragma unroll 1
                    for (int tg = 0; tg < p.tgroups && ok; tg++) {
#pragma unroll 1
                        for (int kq = 0; kq < p.kgroups && ok; kq++, it++) ok = load_stage(c, tg * kTps, r, s, kq);
                        s += kTps;
                        if (s >= p.kw) { s = 0; r++; }
                    }
                }
            }
            if (lane == 0) DLF_TRACE_FLUSH_N(p.status, pacc, 17 + 2 * role, 2);
        }
    } else if (warp == kMmaWarp) {
        // ---- MMA issuer: the whole warp walks the loop (warp-uniform addresses), one elected lane issues ----
        const uint32_t idesc = umma_idesc_f16(p.BN);
        const uint64_t desc0 = umma_desc_sw128(0);
        const uint32_t b_chunk16 = static_cast<uint32_t>(p.BN) * 8u;  // one 64-channel weight slab, in 16-byte units
        const uint32_t a_chunk16 = static_cast<uint32_t>(p.a_bytes) >> 4;  // one 64-channel slab of the tile's pixels (rows rounded up to 8)
        uint32_t it = 0, j = 0, ring_ph = 0;
        int ring_st = 0;   // ring position and phase as counters: no division in the issue loop
        bool ok = true;
        DLF_TRACE_DECL(macc, mmark);  // cycles of CTA 0's issuer: 0 accumulator wait, 1 stage wait, 2 issue
#pragma unroll 1
        for (int t = blockIdx.x; t < p.n_work && ok; t += gridDim.x, j++) {
            const uint32_t acc = j & 1u;
            ok = mbar_wait_warp(&sm.tempty_bar[acc], ((j >> 1) & 1u) ^ 1u, abort_flag, p.status, 0x200 | (blockIdx.x << 12));
            if (!ok) break;
            DLF_TRACE_ACC(macc, 0, mmark);
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + acc * p.acc_stride;
            int kq = 0, k_end = k_iters;
            if (SPLIT) {   // this item's share of the (tap group, K-chunk group) list
                const int l0 = decode_work<SPLIT>(p, t).ks * p.kgs;
                k_end = min(k_iters - l0, p.kgs);
                kq = l0 % p.kgroups;
            }
#pragma unroll 1
            for (int ki = 0; ki < k_end; ki++, it++) {
                const int st = ring_st;
                ok = mbar_wait_warp(&sm.full_bar[st], ring_ph, abort_flag, p.status, 0x300 | (blockIdx.x << 12));
                if (!ok) break;
                if (++ring_st == p.stages) { ring_st = 0; ring_ph ^= 1u; }
                if (it == 0 && lane == 0) DLF_TRACE_POINT(p.status, 3);
                DLF_TRACE_ACC(macc, 1, mmark);
                tc_fence_after_sync();
                const uint32_t sa = base + st * stage_bytes;
                const uint64_t a0 = desc0 + (sa >> 4), b0 = a0 + static_cast<uint32_t>(p.kg * p.a_bytes >> 4);
                const int g_end = min(p.kg, p.kchunks - kq * p.kg);
                if (elect_one()) {
                    if (!ROW) {
#pragma unroll 1
                        for (int g = 0; g < g_end; g++) {
                            const uint64_t ad = a0 + static_cast<uint32_t>(g) * a_chunk16, bd = b0 + static_cast<uint32_t>(g) * b_chunk16;
                            const int ksteps = (kq * p.kg + g == p.kchunks - 1) ? p.ksteps_last : 4;
                            umma_f16(d_tmem, ad, bd, idesc, (ki | g) != 0);
                            if (ksteps > 1) umma_f16(d_tmem, ad + 2, bd + 2, idesc, 1);
                            if (ksteps > 2) umma_f16(d_tmem, ad + 4, bd + 4, idesc, 1);
                            if (ksteps > 3) umma_f16(d_tmem, ad + 6, bd + 6, idesc, 1);
                        }
                    } else {
                        // row mode (whole 64-channel chunks): the three taps of a kernel row read the same window, one
                        // pixel (one 128-byte row) further each
#pragma unroll 1
                        for (int g = 0; g < g_end; g++) {
                            uint64_t ad = a0 + static_cast<uint32_t>(g) * a_chunk16, bd = b0 + static_cast<uint32_t>(g * 3) * b_chunk16;
#pragma unroll
                            for (int sx = 0; sx < 3; sx++, ad += 8, bd += b_chunk16) {
                                umma_f16(d_tmem, ad, bd, idesc, (ki | g | sx) != 0);
                                umma_f16(d_tmem, ad + 2, bd + 2, idesc, 1);
                                umma_f16(d_tmem, ad + 4, bd + 4, idesc, 1);
                                umma_f16(d_tmem, ad + 6, bd + 6, idesc, 1);
                            }
                        }
                    }
                    umma_commit(&sm.empty_bar[st]);  // frees the stage once these MMAs have read it
                }
                __syncwarp();
                DLF_TRACE_ACC(macc, 2, mmark);
                if (++kq == p.kgroups) kq = 0;
            }
            if (ok && elect_one()) umma_commit(&sm.tfull_bar[acc]);
            __syncwarp();
            if (j == 0 && lane == 0) DLF_TRACE_POINT(p.status, 4);
        }
        if (lane == 0) DLF_TRACE_FLUSH_N(p.status, macc, 14, 3);
    } else {
        // ---- epilogue warps ---------------------------------------------------------------------------
        const int q = warp & 3;              // TMEM lane quarter this warp may read
        const int part = warp >> 2;          // which of the interleaved 32-column chunks
        const int m = q * 32 + lane;
        const int tw = m % p.TW, th = (m / p.TW) % p.TH, tn = m / (p.TW * p.TH);
        const int Hp = POOL ? p.Ho / 2 : p.Ho, Wp = POOL ? p.Wo / 2 : p.Wo;
        uint8_t* stage_out = stage0 + p.stage_out_off;
        const bool issuer = (threadIdx.x == 0);
        {   // bias of every output channel, zero past C_out (the channel tile is padded to 16): staged by the epilogue
            // warps alone, after the CTA-wide barrier, so that the producers' first copies do not wait for these loads
            const int n_bias = p.n_tiles_n * p.BN;
#pragma unroll 1
            for (int i = threadIdx.x; i < n_bias; i += 32 * kEpiWarps) bias_s[i] = i < p.Cout ? __ldg(p.bias + i) + (p.bias2 ? __ldg(p.bias2 + i) : 0.0f) : 0.0f;
            asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
        }
        uint32_t j = 0, out_ph = 0;
        int out_b = 0;   // staging buffer of the next tile and the phase of its barriers, as counters
        bool ok = true;
        if (RES && POOL) ok = grid_wait(gs, lane, abort_flag, p.status);   // residual read with plain loads
        DLF_TRACE_DECL(eacc, emark);  // cycles of CTA 0's first epilogue thread: 0 staging-buffer wait, 1 accumulator wait, 2 drain
#pragma unroll 1
        for (int t = blockIdx.x; t < p.n_work && ok; t += gridDim.x, j++) {
            const TileCoord c = decode_work<SPLIT>(p, t);
            const uint32_t acc = j & 1u;
            const int n = c.n0 + tn, ho = c.ho0 + th, wo = c.wo0 + tw;
            const bool valid = m < p.rows && n < p.N && ho < p.Ho && wo < p.Wo;
            const long long pix = (static_cast<long long>(n) * p.Ho + ho) * p.Wo + wo;
            const long long opix = POOL ? (static_cast<long long>(n) * Hp + (ho >> 1)) * Wp + (wo >> 1) : pix;
            const bool writer = valid && (!POOL || (((ho | wo) & 1) == 0 && (ho >> 1) < Hp && (wo >> 1) < Wp));
            const int ncols = min(p.BN, ((p.Cout - c.co0) + 15) & ~15);
            if constexpr (SPLIT) {
                // Split-K: this item's raw fp32 sums go to global memory; of the items of one tile, the warp that
                // arrives last at the (tile, warp) counter adds the shares up in their fixed order (so the result
                // does not depend on which was last), applies bias and activation and writes the fp16 output.
                ok = mbar_wait(&sm.tfull_bar[acc], (j >> 1) & 1u, abort_flag, p.status, 0x400 | (blockIdx.x << 12));
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * p.acc_stride;
                const size_t share = static_cast<size_t>(p.rows) * p.acc_stride;   // floats of one item's partial tile
                float* tile0 = p.partial + static_cast<size_t>(c.tile) * p.splits * share + static_cast<size_t>(min(m, p.rows - 1)) * p.acc_stride;
#pragma unroll 1
                for (int cc = part * 32; cc < ncols; cc += 32 * kEpiParts) {
                    uint32_t r[32];
                    __syncwarp();
                    tmem_ld32_issue(taddr + cc, r);
                    tmem_ld32_wait(r);
                    if (m < p.rows) {
                        float4* dst = reinterpret_cast<float4*>(tile0 + c.ks * share + cc);
#pragma unroll
                        for (int g = 0; g < 8; g++)
                            __stcg(dst + g, make_float4(__uint_as_float(r[4 * g]), __uint_as_float(r[4 * g + 1]), __uint_as_float(r[4 * g + 2]), __uint_as_float(r[4 * g + 3])));
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.tempty_bar[acc]);
                __threadfence();
                __syncwarp();
                int* cnt = p.counters + c.tile * kEpiWarps + warp;
                int old = 0;
                if (lane == 0) old = atomicAdd(cnt, 1);
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old == p.splits - 1) {
                    __threadfence();
                    if (valid) {
#pragma unroll 1
                        for (int cc = part * 32; cc < ncols; cc += 32 * kEpiParts) {
                            const int nc = min(32, ncols - cc);
#pragma unroll
                            for (int g = 0; g < 4; g++) {
                                if (g * 8 >= nc) break;
                                const int co = c.co0 + cc + g * 8;
                                const float4 b0 = *reinterpret_cast<const float4*>(bias_s + co);
                                const float4 b1 = *reinterpret_cast<const float4*>(bias_s + co + 4);
                                float a[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                                const float4* src = reinterpret_cast<const float4*>(tile0 + cc + g * 8);
#pragma unroll 1
                                for (int sp = 0; sp < p.splits; sp++, src += share / 4) {
                                    const float4 v0 = __ldcg(src), v1 = __ldcg(src + 1);
                                    a[0] += v0.x; a[1] += v0.y; a[2] += v0.z; a[3] += v0.w;
                                    a[4] += v1.x; a[5] += v1.y; a[6] += v1.z; a[7] += v1.w;
                                }
                                uint4 o;
                                uint32_t* ou = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                                for (int e = 0; e < 4; e++) {
                                    const __half2 hv = act_h2<ACT>(__floats2half2_rn(a[2 * e], a[2 * e + 1]));
                                    ou[e] = *reinterpret_cast<const uint32_t*>(&hv);
                                }
                                if (co < p.Cout) *reinterpret_cast<uint4*>(p.out + pix * p.Cout + co) = o;
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) *cnt = 0;   // ready for the next launch
                }
                continue;
            }
            // The residual of this pixel's next 32 channels, four 16-byte loads issued together without a
            // branch (clamped address; `rok` keeps which are real): fetched one column pass ahead, the first
            // before the accumulator is even complete, so that their latency is never waited for.
            uint4 rcur[4], rnext[4];
            uint32_t rok = 0u, rok_next = 0u;
            auto res_load = [&](int cc, uint4 (&rv)[4], uint32_t& okm) {
                okm = 0u;
#pragma unroll
                for (int g = 0; g < 4; g++) {
                    const int co = c.co0 + cc + g * 8;
                    const bool okg = valid && cc + g * 8 < ncols && co < p.Cout;
                    rv[g] = __ldg(reinterpret_cast<const uint4*>(p.res + (okg ? pix * p.Cout + co : 0)));
                    okm |= (okg ? 1u : 0u) << g;
                }
            };
            if (RES && POOL) res_load(part * 32, rcur, rok);
            const int sb = out_b;   // this tile's staging buffer; the next tile takes the next one
            const uint32_t sph = out_ph;
            if (++out_b == p.out_bufs) { out_b = 0; out_ph ^= 1u; }
            uint8_t* sout = stage_out + sb * p.out_buf_bytes;
            if (!POOL) {   // the staging buffer is free (first uses pass at once) / holds this tile's residual
                ok = mbar_wait(&sm.sfree_bar[sb], RES ? sph : sph ^ 1u, abort_flag, p.status, 0x600 | (blockIdx.x << 12));
                if (!ok) break;
            }
            DLF_TRACE_ACC(eacc, 0, emark);
            ok = mbar_wait(&sm.tfull_bar[acc], (j >> 1) & 1u, abort_flag, p.status, 0x400 | (blockIdx.x << 12));
            if (!ok) break;
            DLF_TRACE_ACC(eacc, 1, emark);
            if (j == 0 && issuer) DLF_TRACE_POINT(p.status, 5);
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * p.acc_stride;
            // One 32-column chunk of the accumulator row: bias, residual, activation, rounding, store.
            auto drain = [&](const uint32_t (&r)[32], int cc) {
                const int nc = min(32, ncols - cc);
                if (RES && POOL && cc + 32 * kEpiParts < ncols) res_load(cc + 32 * kEpiParts, rnext, rok_next);
#pragma unroll
                for (int g = 0; g < 4; g++) {
                    if (g * 8 >= nc) break;
                    const int co = c.co0 + cc + g * 8;  // first of 8 channels
                    float a[8];
                    const float4 b0 = *reinterpret_cast<const float4*>(bias_s + co);
                    const float4 b1 = *reinterpret_cast<const float4*>(bias_s + co + 4);
                    a[0] = __uint_as_float(r[g * 8 + 0]) + b0.x; a[1] = __uint_as_float(r[g * 8 + 1]) + b0.y; a[2] = __uint_as_float(r[g * 8 + 2]) + b0.z; a[3] = __uint_as_float(r[g * 8 + 3]) + b0.w;
                    a[4] = __uint_as_float(r[g * 8 + 4]) + b1.x; a[5] = __uint_as_float(r[g * 8 + 5]) + b1.y; a[6] = __uint_as_float(r[g * 8 + 6]) + b1.z; a[7] = __uint_as_float(r[g * 8 + 7]) + b1.w;
                    const int g8 = (cc >> 3) + g;
                    uint4* sptr = reinterpret_cast<uint4*>(sout + (g8 >> 3) * kABytes + m * 128 + (((g8 & 7) ^ (m & 7)) << 4));
                    if (RES && !POOL) {   // the residual tile was loaded into the staging buffer (zero outside the tensor)
                        const uint4 rv = *sptr;
                        const __half2* rh = reinterpret_cast<const __half2*>(&rv);
#pragma unroll
                        for (int e = 0; e < 4; e++) {
                            const float2 f = __half22float2(rh[e]);
                            a[2 * e] += f.x;
                            a[2 * e + 1] += f.y;
                        }
                    }
                    if (RES && POOL) {
                        const bool okg = (rok >> g) & 1u;
                        const __half2* rh = reinterpret_cast<const __half2*>(&rcur[g]);
#pragma unroll
                        for (int e = 0; e < 4; e++) {
                            const float2 f = __half22float2(rh[e]);
                            a[2 * e] += okg ? f.x : 0.0f;
                            a[2 * e + 1] += okg ? f.y : 0.0f;
                        }
                    }
                    uint4 o;
                    uint32_t* ou = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                    for (int e = 0; e < 4; e++) {
                        __half2 hv = act_h2<ACT>(__floats2half2_rn(a[2 * e], a[2 * e + 1]));   // (clamped after the rounding: same bits)
                        if (POOL) {  // rounded first, then the max over the 2x2 window held by this warp
                            hv = __hmax2(hv, __shfl_xor_sync(0xffffffffu, hv, 1));
                            hv = __hmax2(hv, __shfl_xor_sync(0xffffffffu, hv, p.TW));
                        }
                        ou[e] = *reinterpret_cast<uint32_t*>(&hv);
                    }
                    if (POOL) {
                        if (writer && co < p.Cout) *reinterpret_cast<uint4*>(p.out + opix * p.Cout + co) = o;
                    } else {
                        *sptr = o;
                    }
                }
                if (RES && POOL) {
#pragma unroll
                    for (int g = 0; g < 4; g++) rcur[g] = rnext[g];
                    rok = rok_next;
                }
            };
#pragma unroll 1
            for (int cc = part * 32; cc < ncols; cc += 32 * kEpiParts) {
                uint32_t r[32];
                __syncwarp();  // the aligned TMEM load needs the whole warp converged
                tmem_ld32_issue(taddr + cc, r);
                tmem_ld32_wait(r);
                drain(r, cc);
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.tempty_bar[acc]);  // the accumulator is drained
            if (!POOL) {
                fence_proxy_async_smem();  // the staging tile is read by the TMA unit
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.sfull_bar[sb]);
            }
            if (j == 0 && issuer) DLF_TRACE_POINT(p.status, 6);
            DLF_TRACE_ACC(eacc, 2, emark);
        }
        if (issuer) DLF_TRACE_FLUSH_N(p.status, eacc, 8, 3);
    }

}

// Initialises the barriers for a ring of `stages` stages (thread 0; `again`: they hold valid objects already).
__device__ __forceinline__ void conv_tc_init_bars(const ConvBars& sm, int stages, bool again) {
    if (again) {
        for (int i = 0; i < 8; i++) { mbar_inval(&sm.full_bar[i]); mbar_inval(&sm.empty_bar[i]); }
        for (int i = 0; i < 2; i++) { mbar_inval(&sm.tfull_bar[i]); mbar_inval(&sm.tempty_bar[i]); }
        for (int i = 0; i < kMaxOutBufs; i++) { mbar_inval(&sm.sfull_bar[i]); mbar_inval(&sm.sfree_bar[i]); }
    }
    for (int i = 0; i < (again ? 8 : stages); i++) {
        mbar_init(&sm.full_bar[i], 2);  // the A and the B producer each arrive with their byte count
        mbar_init(&sm.empty_bar[i], 1);
    }
    for (int i = 0; i < 2; i++) {
        mbar_init(&sm.tfull_bar[i], 1);
        mbar_init(&sm.tempty_bar[i], kEpiWarps);
    }
    for (int i = 0; i < kMaxOutBufs; i++) {
        mbar_init(&sm.sfull_bar[i], kEpiWarps);
        mbar_init(&sm.sfree_bar[i], 1);
    }
    fence_barrier_init();
}

template <int ACT, bool POOL, bool RES, bool ROW, bool SPLIT>
__global__ void __launch_bounds__(kThreads, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tmw,
               const __grid_constant__ CUtensorMap tmy, const __grid_constant__ CUtensorMap tmr,
               const __grid_constant__ CUtensorMap tmx2, const __grid_constant__ CUtensorMap tmw2, const ConvTcParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[8], empty_bar[8], tfull_bar[2], tempty_bar[2];
    __shared__ uint64_t sfull_bar[kMaxOutBufs], sfree_bar[kMaxOutBufs];  // staging buffer: filled by the epilogue / free again (residual landed)
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    if (threadIdx.x == 0) DLF_TRACE_POINT(p.status, 0);
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* stage0 = smem_raw + (base - smem_u32(smem_raw));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const ConvBars sm{full_bar, empty_bar, tfull_bar, tempty_bar, sfull_bar, sfree_bar, &abort_s};

    if (threadIdx.x == 0) {
        abort_s = 0;
        conv_tc_init_bars(sm, p.stages, false);
        tma_prefetch_desc(&tmx);
        tma_prefetch_desc(&tmw);
        if (!POOL) tma_prefetch_desc(&tmy);
        if (!POOL && RES) tma_prefetch_desc(&tmr);
        if (p.kchunks1 < p.kchunks) { tma_prefetch_desc(&tmx2); tma_prefetch_desc(&tmw2); }
    }
    if (warp == kMmaWarp) {
        tmem_alloc(&tmem_base_s, p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();
    // everything above overlapped the previous kernel; from here on its outputs are read - except by the
    // weight producers, which only read constants and may run ahead
    if (warp < kProdWarp0 || warp == kStoreWarp) pdl_wait();   // (the input producers wait once they have decoded their first work item)
    if (threadIdx.x == 0) DLF_TRACE_POINT(p.status, 1);
    const uint32_t tmem_base = tmem_base_s;

    conv_tc_roles<ACT, POOL, RES, ROW, SPLIT>(&tmx, &tmw, &tmy, &tmr, &tmx2, &tmw2, p, sm, tmem_base, stage0, base, GridSync{nullptr, 0u});

    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) {
        if (abort_s) __nanosleep(20000);  // let copies in flight land before the CTA retires
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, p.tmem_cols);
        if (lane == 0) DLF_TRACE_POINT(p.status, 7);
    }
}

// ---- several layers in one launch ------------------------------------------------------------------------------------------
// A fusion group of dense convolutions whose maps are too large (or whose shapes are too irregular: strides, a projection
// branch, a residual from inside the group) to be handed over in shared memory runs as ONE persistent kernel all the same:
// the CTAs walk the group's layers together, separated by a device-wide barrier, and a layer's output goes to its
// workspace slot, which at these sizes stays in the 126 MB L2 until the next layer has read it.  What the group saves
// against one kernel per layer is the kernel boundary (tear-down, launch, set-up, first descriptor fetch: about 5.5 us
// measured, against about 2.5 us for the barrier and the first loads behind it) - the paper's "layers compiled as one block
// on one core count" (Sec. III-B, Sec. IV-C) in the form this chip's cache makes possible.
constexpr int kMaxSeq = 16;
struct SeqLayer {
    CUtensorMap tmx, tmw, tmy, tmr;
    ConvTcParams p;
    int variant;   // ((act * 2 + pool) * 2 + res) * 2 + row
    int pad_[3];
};
struct SeqParams {
    SeqLayer L[kMaxSeq];
    int n_layers;
    unsigned* sync;   // two words, zero between launches: layers finished x CTAs, CTAs done
    int* status;
};

// One layer of a multi-layer launch, as a function of its own: each variant then gets its own register allocation
// instead of the union of all of them inside the calling kernel.
template <int ACT, bool POOL, bool RES, bool ROW>
__device__ __noinline__ void conv_seq_layer(const SeqLayer* Y, const ConvTcParams* p, const ConvBars* sm, uint32_t tmem_base, uint8_t* stage0,
                                            uint32_t base, unsigned* sync, unsigned target) {
    conv_tc_roles<ACT, POOL, RES, ROW, false>(&Y->tmx, &Y->tmw, &Y->tmy, &Y->tmr, &Y->tmx, &Y->tmw, *p, *sm, tmem_base, stage0, base, GridSync{sync, target});
}

__global__ void __launch_bounds__(kThreads, 1) conv_seq_kernel(const __grid_constant__ SeqParams sp) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[8], empty_bar[8], tfull_bar[2], tempty_bar[2];
    __shared__ uint64_t sfull_bar[kMaxOutBufs], sfree_bar[kMaxOutBufs];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    // the current layer's parameters, copied out of the kernel's parameter block: the roles read them all the time, and a
    // dynamically indexed parameter array is read through generic loads
    __shared__ __align__(16) ConvTcParams p_s;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* stage0 = smem_raw + (base - smem_u32(smem_raw));
    const int warp = threadIdx.x >> 5;
    const ConvBars sm{full_bar, empty_bar, tfull_bar, tempty_bar, sfull_bar, sfree_bar, &abort_s};

    if (threadIdx.x == 0) {
        abort_s = 0;
        conv_tc_init_bars(sm, 8, false);
    }
    if (warp == kMmaWarp) {
        tmem_alloc(&tmem_base_s, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_s;

#pragma unroll 1
    for (int l = 0; l < sp.n_layers; l++) {
        const SeqLayer& Y = sp.L[l];
        if (l == 1 && threadIdx.x == 0) DLF_TRACE_POINT(sp.status, 20);
        for (int i = threadIdx.x; i < static_cast<int>(sizeof(ConvTcParams) / 4); i += kThreads)
            reinterpret_cast<int*>(&p_s)[i] = reinterpret_cast<const int*>(&Y.p)[i];
        if (threadIdx.x == 0) {   // fresh barriers for this layer's ring (every role is past the previous layer: see the barrier below)
            if (l > 0) conv_tc_init_bars(sm, 8, true);
            tma_prefetch_desc(&Y.tmx);
            tma_prefetch_desc(&Y.tmw);
        }
        __syncthreads();
        if (l == 1 && threadIdx.x == 0) DLF_TRACE_POINT(sp.status, 21);
        const unsigned target = static_cast<unsigned>(l) * gridDim.x;   // every CTA has finished the layers before this one
#define DLF_SEQ_CASE(ACT, POOL, RES, ROW)                                                                      \
    case ((ACT * 2 + POOL) * 2 + RES) * 2 + ROW:                                                               \
        conv_seq_layer<ACT, POOL != 0, RES != 0, ROW != 0>(&Y, &p_s, &sm, tmem_base, stage0, base, sp.sync, target); \
        break;
        switch (Y.variant) {
            DLF_SEQ_CASE(0, 0, 0, 0) DLF_SEQ_CASE(0, 0, 0, 1) DLF_SEQ_CASE(0, 0, 1, 0) DLF_SEQ_CASE(0, 0, 1, 1) DLF_SEQ_CASE(0, 1, 0, 0) DLF_SEQ_CASE(0, 1, 1, 0)
            DLF_SEQ_CASE(1, 0, 0, 0) DLF_SEQ_CASE(1, 0, 0, 1) DLF_SEQ_CASE(1, 0, 1, 0) DLF_SEQ_CASE(1, 0, 1, 1) DLF_SEQ_CASE(1, 1, 0, 0) DLF_SEQ_CASE(1, 1, 1, 0)
            DLF_SEQ_CASE(2, 0, 0, 0) DLF_SEQ_CASE(2, 0, 0, 1) DLF_SEQ_CASE(2, 0, 1, 0) DLF_SEQ_CASE(2, 0, 1, 1) DLF_SEQ_CASE(2, 1, 0, 0) DLF_SEQ_CASE(2, 1, 1, 0)
            default: break;
        }
#undef DLF_SEQ_CASE
        // the layer is finished on this CTA once its stores have completed and every role has left it
        if (l == 0 && threadIdx.x == 0) DLF_TRACE_POINT(sp.status, 22);
        if (l == 0 && threadIdx.x == 32 * kStoreWarp) DLF_TRACE_POINT(sp.status, 23);
        if (warp == kStoreWarp) {
            tma_store_wait_all();
            asm volatile("fence.proxy.async;" ::: "memory");
        }
        if (l == 0 && threadIdx.x == 32 * kStoreWarp) DLF_TRACE_POINT(sp.status, 24);
        __threadfence();
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
        if (l == 0 && threadIdx.x == 0) DLF_TRACE_POINT(sp.status, 25);
        if (threadIdx.x == 0 && l + 1 < sp.n_layers) {
            __threadfence();
            atomicAdd(sp.sync, 1u);
        }
        if (l == 0 && threadIdx.x == 0) DLF_TRACE_POINT(sp.status, 26);
    }
    // the last CTA to leave puts the two counters back to zero for the next launch
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(sp.sync + 1, 1u) == gridDim.x - 1) {
            sp.sync[0] = 0u;
            sp.sync[1] = 0u;
            __threadfence();
        }
    }
    if (warp == kMmaWarp) {
        if (abort_s) __nanosleep(20000);
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

struct Tile {
    int tw, th, tn;
};

// Pixel tile TN x TH x TW of at most 128 output pixels (the UMMA's M): the fewest tiles, then the fewest
// rows (rows past TN * TH * TW are neither loaded nor stored: an image smaller than a power-of-two tile
// costs no shared-memory fill), then the widest.  The pooled epilogue reduces 2x2 windows with warp
// shuffles and keeps power-of-two tiles of 128 pixels.
Tile pick_tile(int N, int Ho, int Wo, int pool) {
    Tile best{16, 8, 1};
    long long best_tiles = -1;
    if (pool) {
        for (int tw = 16; tw >= 2; tw >>= 1)
            for (int th = 128 / tw; th >= 2; th >>= 1) {
                const int tn = 128 / (tw * th);
                const long long tiles = static_cast<long long>((Wo + tw - 1) / tw) * ((Ho + th - 1) / th) * ((N + tn - 1) / tn);
                if (best_tiles < 0 || tiles < best_tiles) {
                    best_tiles = tiles;
                    best = Tile{tw, th, tn};
                }
            }
        return best;
    }
    int best_rows = 0;
    for (int tn = 1; tn <= std::min(N, 128); tn++)
        for (int th = 1; th <= std::min(Ho, 128 / tn); th++) {
            const int tw_max = std::min(Wo, 128 / (tn * th));
            const int tw = (Wo + (Wo + tw_max - 1) / tw_max - 1) / ((Wo + tw_max - 1) / tw_max);  // as many tiles per row, evenly wide
            const int rows = tn * th * tw;
            const long long tiles = static_cast<long long>((Wo + tw - 1) / tw) * ((Ho + th - 1) / th) * ((N + tn - 1) / tn);
            if (best_tiles < 0 || tiles < best_tiles || (tiles == best_tiles && (rows < best_rows || (rows == best_rows && tw > best.tw)))) {
                best_tiles = tiles;
                best_rows = rows;
                best = Tile{tw, th, tn};
            }
        }
    return best;
}

typedef void (*KernelFn)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap,
                         const ConvTcParams);

template <int ACT, bool POOL, bool RES>
KernelFn pick_row(bool row) {
    if constexpr (POOL) return conv_tc_kernel<ACT, POOL, RES, false, false>;   // the row mode has no pooled epilogue
    else return row ? conv_tc_kernel<ACT, POOL, RES, true, false> : conv_tc_kernel<ACT, POOL, RES, false, false>;
}
template <int ACT, bool POOL>
KernelFn pick_res(bool res, bool row) {
    return res ? pick_row<ACT, POOL, true>(row) : pick_row<ACT, POOL, false>(row);
}
template <int ACT>
KernelFn pick_pool(bool pool, bool res, bool row) {
    return pool ? pick_res<ACT, true>(res, row) : pick_res<ACT, false>(res, row);
}
// split-K variants: layers without pooling or residual
template <int ACT>
KernelFn pick_split_row(bool row) {
    return row ? conv_tc_kernel<ACT, false, false, true, true> : conv_tc_kernel<ACT, false, false, false, true>;
}
KernelFn pick_split(int act, bool row) {
    if (act == 0) return pick_split_row<0>(row);
    if (act == 1) return pick_split_row<1>(row);
    return pick_split_row<2>(row);
}
KernelFn pick_kernel(int act, bool pool, bool res, bool row) {
    if (act == 0) return pick_pool<0>(pool, res, row);
    if (act == 1) return pick_pool<1>(pool, res, row);
    return pick_pool<2>(pool, res, row);
}

}  // namespace

bool conv_tc_supported(const ConvArgs& a) {
    if (a.groups != 1) return false;
    if (a.Cin < 8 || a.Cout < 8 || a.Cin % 8 || a.Cout % 8 || a.Cout > 4096) return false;
    if (a.stride < 1 || a.stride > 2) return false;
    if (a.kh * a.kw > 49) return false;
    if (a.N < 1 || a.Ho < 1 || a.Wo < 1) return false;
    return true;
}

// The second source joins a 1x1 stride-1 layer chunk by chunk of 64 channels; both channel counts are whole chunks.
bool conv_tc_dual_supported(const ConvArgs& a) {
    if (!conv_tc_supported(a)) return false;
    if (a.kh != 1 || a.kw != 1 || a.stride != 1 || a.pad != 0 || a.pool) return false;
    if (a.Cin % 64 || a.Cin2 < 64 || a.Cin2 % 64) return false;
    if (a.stride2 < 1 || a.stride2 > 2) return false;
    if (a.H2 < 1 || a.W2 < 1 || (a.H2 - 1) / a.stride2 + 1 != a.Ho || (a.W2 - 1) / a.stride2 + 1 != a.Wo) return false;
    return true;
}

namespace {
// Everything a launch of one layer needs: tensor maps, parameters, the kernel variant, shared memory, grid.
struct ConvTcLaunch {
    CUtensorMap tmx, tmw, tmy, tmr, tmx2, tmw2;
    ConvTcParams p;
    int act, pool, res, row, split;
    size_t smem;
    int grid;
};

int conv_tc_prepare(const ConvArgs& a_in, int sm_count, int* status_dev, ConvTcLaunch* out) {
    if (!conv_tc_supported(a_in)) return DLF_E_UNSUPPORTED;
    const bool dual = a_in.x2 != nullptr;
    if (dual && !conv_tc_dual_supported(a_in)) return DLF_E_UNSUPPORTED;
    // A 1x1 stride-1 convolution has no spatial structure: its N x H x W pixels are one list, cut into tiles of any
    // length, so that the persistent grid's rounds can be filled evenly (below) whatever the image size.
    ConvArgs a = a_in;
    const long long flat_pixels = static_cast<long long>(a_in.N) * a_in.H * a_in.W;
    // (measured to pay for the output-bound layers with few input channels; with more, the image-shaped tiles were as fast or faster)
    const bool flat = a.kh == 1 && a.kw == 1 && a.stride == 1 && a.pad == 0 && !a.pool && flat_pixels < (1ll << 31) && (a.Cin <= 128 || a.H * a.W == 1) && !dual;
    if (flat) {
        a.N = 1; a.H = 1; a.Ho = 1;
        a.W = a.Wo = static_cast<int>(flat_pixels);
    }
    ConvTcParams p{};
    p.N = a.N; p.Ho = a.Ho; p.Wo = a.Wo; p.Cout = a.Cout;
    p.kh = a.kh; p.kw = a.kw; p.stride = a.stride; p.pad = a.pad;
    const int cout16 = (a.Cout + 15) / 16 * 16;
    p.kchunks = (a.Cin + 63) / 64;
    p.ksteps_last = ((a.Cin - (p.kchunks - 1) * 64) + 15) / 16;
    p.kchunks1 = p.kchunks;
    if (dual) {   // the second source's chunks follow the first's in K
        p.kchunks += a.Cin2 / 64;
        p.stride2 = a.stride2;
    }
    p.grouped = (a.Cin % 64 == 0) ? 1 : 0;
    Tile tl{};
    long long m_tiles = 0;
    int bias_bytes = 0;
    int splits = 1;   // split-K shares per tile that configure() lays the channel tiles out for
    auto set_tile = [&](const Tile& t, int taps_per_stage) {
        tl = t;
        p.TW = tl.tw; p.TH = tl.th; p.TN = tl.tn;
        p.rows = tl.tw * tl.th * tl.tn;
        p.a_bytes = (p.rows + 7) / 8 * 8 * 128;
        p.tiles_w = (a.Wo + tl.tw - 1) / tl.tw;
        p.tiles_h = (a.Ho + tl.th - 1) / tl.th;
        p.tiles_n = (a.N + tl.tn - 1) / tl.tn;
        p.tps = taps_per_stage;
        p.tgroups = a.kh * a.kw / taps_per_stage;
        m_tiles = static_cast<long long>(p.tiles_w) * p.tiles_h * p.tiles_n;
    };
    // Lays out the ring, the staging buffers and the bias for a shared-memory budget and a widest channel tile;
    // false if not even `min_stages` ring stages (or all of the tile's loads) fit.
    auto configure = [&](int budget, int bn_max, int min_stages) {
        // Channel tile: layers with few pixel tiles (small images, small batch) get narrower channel tiles so
        // that the work list covers the SMs; cost = waves x (tile width + a fixed per-item overhead).  With
        // several channel tiles the width is a multiple of 64, so that a tile's 64-channel TMA store boxes
        // never reach into its neighbour's channels.
        long long best_cost = -1;
        for (int bn : {256, 192, 128, 64}) {
            if (bn > bn_max) continue;
            const int width = std::min(bn, cout16);
            const int nt = (cout16 + width - 1) / width;
            if (nt > 1 && width % 64) continue;
            const long long waves = (m_tiles * nt * splits + sm_count - 1) / sm_count;
            const long long cost = waves * (width + 96);
            if (best_cost < 0 || cost < best_cost) {
                best_cost = cost;
                p.BN = width;
                p.n_tiles_n = nt;
            }
        }
        if (best_cost < 0) return false;
        const int out_planes = (a.pool || splits > 1) ? 0 : (p.BN + 63) / 64;   // (split-K tiles are not staged)
        bias_bytes = (p.n_tiles_n * p.BN * 4 + 1023) / 1024 * 1024;
        p.out_buf_bytes = out_planes * kABytes;
        const int b_bytes = p.tps * p.BN * 128;   // the weight slabs of one 64-channel chunk in a stage
        const int loads_min = p.tgroups * p.kchunks;
        // Two staging buffers (the stores of one tile drain while the next is written) where the ring keeps
        // three stages, or as many as the tile has loads, beside them; else one.
        // (a layer of short tiles - one or two loads each - is bound by the latency of its stores: up to four buffers)
        for (p.out_bufs = a.pool ? 1 : (loads_min <= 2 ? kMaxOutBufs : 2); p.out_bufs >= 1; p.out_bufs--) {
            // the UMMA always reads 128 rows of a slab (two more in the row mode): behind a shorter one it reads on
            // into whatever follows (those accumulator rows are never stored), which must still be this CTA's
            // shared memory
            const int fixed = p.out_bufs * p.out_buf_bytes + bias_bytes + 1024 + (kABytes + 256 - p.a_bytes);
            // K chunks per ring stage: every stage costs the issuing threads a fixed handshake (barrier wait,
            // TMA issue, commit), so a stage carries as many 64-channel chunks as leave room for >= 2 stages
            p.kg = 1;
            if (p.grouped)
                for (int kg : {8, 4, 2})
                    if (kg <= p.kchunks && (kg < 8 || p.rows <= 32) && 2 * kg * (p.a_bytes + b_bytes) <= budget - fixed && (kg == 2 || 3 * kg * (p.a_bytes + b_bytes) <= budget - fixed || p.tgroups * ((p.kchunks + kg - 1) / kg) <= 2)) {
                        p.kg = kg;
                        break;
                    }
            p.kgroups = (p.kchunks + p.kg - 1) / p.kg;
            const int stage_bytes = p.kg * (p.a_bytes + b_bytes);
            p.stages = std::min(8, (budget - fixed) / stage_bytes);
            const int loads = p.tgroups * p.kgroups;
            // (the ring runs on across work items: a tile with one or two loads still wants four stages, so that the
            // next tiles' copies are in flight while this one is multiplied and drained)
            p.stages = std::min(p.stages, std::max(loads, 4));
            p.stage_out_off = p.stages * stage_bytes;
            p.bias_off = p.stage_out_off + p.out_bufs * p.out_buf_bytes;
            if (p.stages >= 1 && (p.out_bufs == 1 || p.stages >= std::min(3, std::max(loads, p.out_bufs)))) break;
        }
        return p.stages >= std::min(min_stages, loads_min);
    };
    // What a CTA streams from L2 into shared memory over the kernel (the bound of the 3x3 layers): waves x bytes per item.
    auto stream_cost = [&]() {
        const long long waves = (m_tiles * p.n_tiles_n + sm_count - 1) / sm_count;
        return static_cast<double>(waves) * p.tgroups * p.kchunks * (p.a_bytes + p.tps * p.BN * 128);
    };
    // Cost of the current layout with `sp` split-K shares per tile: rounds of the grid x cost of a work item, in bytes of
    // shared-memory fill.  An item is bound by the slower of its fill and its UMMAs (measured per M = 128, K = 16
    // instruction: max(N / 2, 32 + N / 4) cycles, against 74 bytes per cycle of fill), plus what it writes (and reads as
    // residual) weighted by the ratio of an SM's fill rate to its share of the HBM rate, plus a fixed hand-off cost; sharing
    // a tile costs the fp32 partial tile's round trip and a hand-over on top.  Negative: `sp` shares are not possible.
    const bool can_split = a.splitk_ws && a.splitk_bytes > kSplitCounterBytes && !a.res && !a.pool && !dual;
    auto split_score = [&](int sp) -> long long {
        const int loads = p.tgroups * p.kgroups;
        const int per = (loads + sp - 1) / sp;
        const long long tiles = m_tiles * p.n_tiles_n;
        const int acc_stride = (p.BN + 31) / 32 * 32;
        if (sp > 1 && (!can_split || (sp - 1) * per >= loads || per * p.kg * p.tps < 8 || tiles * kEpiWarps * 4 > static_cast<long long>(kSplitCounterBytes) ||
                       static_cast<unsigned long long>(tiles) * sp * p.rows * acc_stride * 4 > a.splitk_bytes - kSplitCounterBytes))
            return -1;
        const long long rounds = (tiles * sp + sm_count - 1) / sm_count;
        const long long k_item = std::min<long long>(static_cast<long long>(p.tgroups) * p.kchunks, static_cast<long long>(per) * p.kg);   // 64-channel chunk loads
        const long long fill = k_item * (p.a_bytes + p.tps * p.BN * 128);
        const long long mma = k_item * p.tps * 4 * std::max(p.BN / 2, 32 + p.BN / 4) * 74;
        const long long item = std::max(fill, mma) + static_cast<long long>(p.rows) * p.BN * 2 * (a.res ? 2 : 1) * 27 / 10 +
                               (sp > 1 ? static_cast<long long>(p.rows) * p.BN * 8 * 27 / 10 + 600000 : 0) + 40960;
        return rounds * item;
    };
    // Row mode (3x3, stride 1, pad 1): a tile is TH whole output rows seen with a pitch of Wo + 2, pixel-linear like
    // its input window, so that the three taps of a kernel row read ONE loaded window through descriptors that
    // start 0, 1 and 2 pixels (128-byte rows) into it: the window is streamed 3 times per 64-channel chunk instead of
    // 9 and a stage carries a kernel row's three weight slabs.  The two columns past the image come out as garbage
    // that the epilogue masks and the clipped TMA store never writes.
    bool row_mode = false;
    ConvTcParams p_row{};
    Tile tl_row{};
    int bias_row = 0;
    double cost_row = 0.0;
    if (g_conv_row_mode > 0 && a.kh == 3 && a.kw == 3 && a.stride == 1 && a.pad == 1 && !a.pool && p.grouped && a.Wo + 2 <= 128 && a.W == a.Wo && a.H == a.Ho) {
        const int th_row = std::min(a.Ho, 128 / (a.Wo + 2));
        // several whole images per tile where they fit (an image's rows stay together, so the shifted reads of its
        // valid pixels never reach the next image)
        const int tn_row = th_row == a.Ho ? std::max(1, std::min(a.N, 128 / (th_row * (a.Wo + 2)))) : 1;
        set_tile(Tile{a.Wo + 2, th_row, tn_row}, 3);
        if (configure(kMaxSmem, 128, 2)) {
            row_mode = true;
            p_row = p; tl_row = tl; bias_row = bias_bytes; cost_row = stream_cost();
        }
    }
    if (flat) {
        // tile length: the least (rounds of the grid) x (cost of an item); an item costs what it streams into shared
        // memory (pixels and weight slab per 64-channel chunk) plus what it writes (and reads as residual), the
        // latter weighted by the ratio of an SM's fill rate to its share of the HBM rate, plus a fixed hand-off cost;
        // the channel-tile width follows from the tile count as for every layer.
        // Split-K (few tiles, long K: fully connected layers at small batch, where one work item per tile would leave
        // SMs idle and be bound by the UMMA issue rate): a tile's K range is shared out over `splits` work items that
        // leave fp32 partial tiles in the caller's workspace; chosen together with the tile length.
        int best_r = 0, best_s = 1;
        long long best_score = -1;
        for (int r = 128; r >= 32; r--) {
            for (int sp : {1, 2, 3, 4, 6, 8, 12, 16}) {
                if (sp > 1 && !can_split) break;
                splits = sp;
                set_tile(Tile{std::min(r, a.Wo), 1, 1}, 1);
                if (!configure(kMaxSmem, 256, 1)) continue;
                const long long score = split_score(sp);
                if (score < 0) continue;
                if (best_score < 0 || score < best_score) {
                    best_score = score;
                    best_r = p.rows;
                    best_s = sp;
                }
            }
            if (a.Wo <= r) break;
        }
        if (best_r == 0) return DLF_E_UNSUPPORTED;
        splits = best_s;
        set_tile(Tile{best_r, 1, 1}, 1);
    } else {
        set_tile(pick_tile(a.N, a.Ho, a.Wo, a.pool), 1);
    }
    if (!configure(kMaxSmem, 256, 1)) return DLF_E_UNSUPPORTED;
    if (row_mode && (g_conv_row_mode > 1 || cost_row < 0.8 * stream_cost())) {
        const long long keep_m = static_cast<long long>(p_row.tiles_w) * p_row.tiles_h * p_row.tiles_n;
        p = p_row; tl = tl_row; bias_bytes = bias_row; m_tiles = keep_m;
    }
    if (!flat && can_split && m_tiles * p.n_tiles_n * 2 <= sm_count) {
        // few work items (small images at small batch): share each tile's (tap, K-chunk) list out as well
        const bool row = p.tps == 3;
        const ConvTcParams keep = p;
        const int keep_bias = bias_bytes;
        int best_s = 1;
        long long best_score = -1;
        for (int sp : {1, 2, 3, 4, 6, 8, 12, 16}) {
            splits = sp;
            if (!configure(kMaxSmem, row ? 128 : 256, row ? 2 : 1)) continue;
            const long long score = split_score(sp);
            if (score >= 0 && (best_score < 0 || score < best_score)) {
                best_score = score;
                best_s = sp;
            }
        }
        splits = best_s;
        if (best_s == 1 || !configure(kMaxSmem, row ? 128 : 256, row ? 2 : 1)) {
            splits = 1;
            p = keep;
            bias_bytes = keep_bias;
        }
    }
    // stores in flight: all buffers but one where a buffer also has to take the next tile's residual in time
    p.store_depth = std::max(1, a.res ? p.out_bufs - 1 : p.out_bufs);
    p.splits = splits;
    p.kgs = (p.tgroups * p.kgroups + splits - 1) / splits;
    if (splits > 1) {
        p.counters = static_cast<int*>(a.splitk_ws);
        p.partial = reinterpret_cast<float*>(static_cast<uint8_t*>(a.splitk_ws) + kSplitCounterBytes);
    }
    const long long n_work = static_cast<long long>(p.tiles_w) * p.tiles_h * p.tiles_n * p.n_tiles_n * splits;
    if (n_work > 0x7fffffffLL) return DLF_E_UNSUPPORTED;
    p.n_work = static_cast<int>(n_work);
    uint32_t cols = 32;
    p.acc_stride = (p.BN + 31) / 32 * 32;
    while (cols < static_cast<uint32_t>(2 * p.acc_stride)) cols <<= 1;
    p.tmem_cols = cols;
    p.bias = a.bias; p.bias2 = dual ? a.bias2 : nullptr; p.res = static_cast<const __half*>(a.res); p.out = static_cast<__half*>(a.y);
    p.status = status_dev;

    CUtensorMap tmx, tmw, tmy, tmr, tmx2, tmw2;
    const uint64_t taps64 = static_cast<uint64_t>(a.kh) * a.kw;
    if (p.grouped) {
        // input seen as (64 channels, W, H, N, C_in / 64): one box carries one 64-channel chunk of a tap's window
        const uint64_t dims[5] = {64, static_cast<uint64_t>(a.W), static_cast<uint64_t>(a.H), static_cast<uint64_t>(a.N),
                                  static_cast<uint64_t>(a.Cin / 64)};
        const uint64_t strides[4] = {static_cast<uint64_t>(a.Cin) * 2, static_cast<uint64_t>(a.W) * a.Cin * 2,
                                     static_cast<uint64_t>(a.H) * a.W * a.Cin * 2, 128};
        const uint32_t box[5] = {64, static_cast<uint32_t>(tl.tw * a.stride), static_cast<uint32_t>(tl.th * a.stride),
                                 static_cast<uint32_t>(tl.tn), 1};
        const uint32_t es[5] = {1, static_cast<uint32_t>(a.stride), static_cast<uint32_t>(a.stride), 1, 1};
        int rc = encode_tmap(&tmx, a.x, 5, dims, strides, box, es);
        if (rc) return rc;
        // weights [cout][tap][cin] seen as (64 channels, cout, tap, C_in / 64)
        const uint64_t wdims[4] = {64, static_cast<uint64_t>(a.Cout), taps64, static_cast<uint64_t>(a.Cin / 64)};
        const uint64_t wstrides[3] = {taps64 * a.Cin * 2, static_cast<uint64_t>(a.Cin) * 2, 128};
        const uint32_t wbox[4] = {64, static_cast<uint32_t>(p.BN), static_cast<uint32_t>(p.tps), 1};
        const uint32_t wes[4] = {1, 1, 1, 1};
        rc = encode_tmap(&tmw, a.w, 4, wdims, wstrides, wbox, wes);
        if (rc) return rc;
    } else {
        const uint64_t dims[4] = {static_cast<uint64_t>(a.Cin), static_cast<uint64_t>(a.W), static_cast<uint64_t>(a.H),
                                  static_cast<uint64_t>(a.N)};
        const uint64_t strides[3] = {static_cast<uint64_t>(a.Cin) * 2, static_cast<uint64_t>(a.W) * a.Cin * 2,
                                     static_cast<uint64_t>(a.H) * a.W * a.Cin * 2};
        const uint32_t box[4] = {64, static_cast<uint32_t>(tl.tw * a.stride), static_cast<uint32_t>(tl.th * a.stride),
                                 static_cast<uint32_t>(tl.tn)};
        const uint32_t es[4] = {1, static_cast<uint32_t>(a.stride), static_cast<uint32_t>(a.stride), 1};
        int rc = encode_tmap(&tmx, a.x, 4, dims, strides, box, es);
        if (rc) return rc;
        const uint64_t wdims[3] = {static_cast<uint64_t>(a.Cin), taps64, static_cast<uint64_t>(a.Cout)};
        const uint64_t wstrides[2] = {static_cast<uint64_t>(a.Cin) * 2, taps64 * a.Cin * 2};
        const uint32_t wbox[3] = {64, 1, static_cast<uint32_t>(p.BN)};
        const uint32_t wes[3] = {1, 1, 1};
        rc = encode_tmap(&tmw, a.w, 3, wdims, wstrides, wbox, wes);
        if (rc) return rc;
    }
    tmx2 = tmx; tmw2 = tmw;
    if (dual) {   // the second source, seen like the first: (64 channels, W2, H2, N, Cin2 / 64) read with its own stride
        const uint64_t dims[5] = {64, static_cast<uint64_t>(a.W2), static_cast<uint64_t>(a.H2), static_cast<uint64_t>(a.N),
                                  static_cast<uint64_t>(a.Cin2 / 64)};
        const uint64_t strides[4] = {static_cast<uint64_t>(a.Cin2) * 2, static_cast<uint64_t>(a.W2) * a.Cin2 * 2,
                                     static_cast<uint64_t>(a.H2) * a.W2 * a.Cin2 * 2, 128};
        const uint32_t box[5] = {64, static_cast<uint32_t>(tl.tw * a.stride2), static_cast<uint32_t>(tl.th * a.stride2),
                                 static_cast<uint32_t>(tl.tn), 1};
        const uint32_t es[5] = {1, static_cast<uint32_t>(a.stride2), static_cast<uint32_t>(a.stride2), 1, 1};
        int rc = encode_tmap(&tmx2, a.x2, 5, dims, strides, box, es);
        if (rc) return rc;
        const uint64_t wdims[4] = {64, static_cast<uint64_t>(a.Cout), 1, static_cast<uint64_t>(a.Cin2 / 64)};
        const uint64_t wstrides[3] = {static_cast<uint64_t>(a.Cin2) * 2, static_cast<uint64_t>(a.Cin2) * 2, 128};
        const uint32_t wbox[4] = {64, static_cast<uint32_t>(p.BN), 1, 1};
        const uint32_t wes[4] = {1, 1, 1, 1};
        rc = encode_tmap(&tmw2, a.w2, 4, wdims, wstrides, wbox, wes);
        if (rc) return rc;
    }
    {   // output map (unused by the pooled variant, which stores from registers)
        const int Hy = a.pool ? a.Ho / 2 : a.Ho, Wy = a.pool ? a.Wo / 2 : a.Wo;
        const uint64_t dims[4] = {static_cast<uint64_t>(a.Cout), static_cast<uint64_t>(Wy), static_cast<uint64_t>(Hy),
                                  static_cast<uint64_t>(a.N)};
        const uint64_t strides[3] = {static_cast<uint64_t>(a.Cout) * 2, static_cast<uint64_t>(Wy) * a.Cout * 2,
                                     static_cast<uint64_t>(Hy) * Wy * a.Cout * 2};
        const uint32_t box[4] = {64, static_cast<uint32_t>(tl.tw), static_cast<uint32_t>(tl.th), static_cast<uint32_t>(tl.tn)};
        const uint32_t es[4] = {1, 1, 1, 1};
        int rc = encode_tmap(&tmy, a.y, 4, dims, strides, box, es);
        if (rc) return rc;
        tmr = tmy;
        if (a.res && !a.pool) {   // the residual has the output's shape
            rc = encode_tmap(&tmr, a.res, 4, dims, strides, box, es);
            if (rc) return rc;
        }
    }
    out->grid = std::max(1, std::min(sm_count, p.n_work));
    // never two of these CTAs on an SM: each may hold all of tensor memory
    out->smem = std::max<size_t>(static_cast<size_t>(p.bias_off) + bias_bytes + 1024 + (kABytes + 256 - p.a_bytes), 120 * 1024);
#ifdef DLF_TRACE
    fprintf(stderr, "conv_tc: tile %dx%dx%d rows %d BN %d x %d splits %d kgs %d kg %d kgroups %d stages %d out_bufs %d work %d grid %d\n", tl.tn, tl.th, tl.tw,
            p.rows, p.BN, p.n_tiles_n, p.splits, p.kgs, p.kg, p.kgroups, p.stages, p.out_bufs, p.n_work, out->grid);
#endif
    out->tmx = tmx; out->tmw = tmw; out->tmy = tmy; out->tmr = tmr; out->tmx2 = tmx2; out->tmw2 = tmw2;
    out->p = p;
    out->act = a.act; out->pool = a.pool != 0; out->res = a.res != nullptr; out->row = p.tps == 3; out->split = splits > 1;
    return DLF_OK;
}
}  // namespace

int launch_conv_tc(const ConvArgs& a, int sm_count, int* status_dev, cudaStream_t s) {
    int rc = conv_tc_init();
    if (rc) return rc;
    ConvTcLaunch L;
    rc = conv_tc_prepare(a, sm_count, status_dev, &L);
    if (rc) return rc;
    const KernelFn fn = L.split ? pick_split(L.act, L.row != 0) : pick_kernel(L.act, L.pool != 0, L.res != 0, L.row != 0);
    cudaError_t e = launch_kernel(fn, L.grid, kThreads, L.smem, s, L.tmx, L.tmw, L.tmy, L.tmr, L.tmx2, L.tmw2, L.p);
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

int g_seq_cooperative = 0;
bool conv_seq_layer_supported(const ConvArgs& a) { return conv_tc_supported(a); }
int conv_seq_max_layers() { return kMaxSeq; }

// Several dense convolutions as one persistent kernel on `sm_count` CTAs (a cooperative launch: every CTA must be resident,
// they wait for one another between the layers).  `sync_dev`: two words of device memory that are zero between launches.
int launch_conv_seq(const ConvArgs* layers, int n_layers, int sm_count, int* status_dev, unsigned* sync_dev, cudaStream_t s) {
    if (n_layers < 1 || n_layers > kMaxSeq || !sync_dev) return DLF_E_PLAN;
    int rc = conv_tc_init();
    if (rc) return rc;
    static SeqParams sp;   // (large: not on the stack; the launch copies it)
    std::memset(&sp, 0, sizeof(sp));
    size_t smem = 0;
    for (int l = 0; l < n_layers; l++) {
        ConvArgs a = layers[l];
        a.splitk_ws = nullptr;   // no split reductions inside a multi-layer launch
        a.splitk_bytes = 0;
        ConvTcLaunch L;
        rc = conv_tc_prepare(a, sm_count, status_dev, &L);
        if (rc) return rc;
        if (L.split || (L.pool && L.row) || a.x2) return DLF_E_UNSUPPORTED;
        SeqLayer& Y = sp.L[l];
        Y.tmx = L.tmx; Y.tmw = L.tmw; Y.tmy = L.tmy; Y.tmr = L.tmr;
        Y.p = L.p;
        Y.variant = ((L.act * 2 + L.pool) * 2 + L.res) * 2 + L.row;
        smem = std::max(smem, L.smem);
    }
    sp.n_layers = n_layers;
    sp.sync = sync_dev;
    sp.status = status_dev;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(sm_count));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_seq_cooperative ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, conv_seq_kernel, sp);
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

int conv_tc_init() {
    static bool attr_set[kMaxDevices] = {};
    const int dev = current_device_slot();
    if (dev < 0) return DLF_E_UNSUPPORTED;
    if (!attr_set[dev]) {
        for (int act = 0; act < 3; act++)
            for (int pool = 0; pool < 2; pool++)
                for (int res = 0; res < 2; res++)
                    for (int row = 0; row < (pool ? 1 : 2); row++) {
                        cudaError_t e = cudaFuncSetAttribute(pick_kernel(act, pool != 0, res != 0, row != 0),
                                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
                        if (e != cudaSuccess) return cuda_fail(e);
                    }
        for (int act = 0; act < 3; act++)
            for (int row = 0; row < 2; row++) {
                cudaError_t e = cudaFuncSetAttribute(pick_split(act, row != 0), cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
                if (e != cudaSuccess) return cuda_fail(e);
            }
        {
            cudaError_t e = cudaFuncSetAttribute(conv_seq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
            if (e != cudaSuccess) return cuda_fail(e);
        }
        attr_set[dev] = true;
    }
    return DLF_OK;
}

}  // namespace dlf
