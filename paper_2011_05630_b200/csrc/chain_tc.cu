// Fused fusion-group kernel: a chain of stride-1, size-keeping dense convolutions (3x3 pad 1 or
// 1x1) with bias / activation after each, optional residual and 2x2 max-pool on the last one,
// executed by ONE kernel whose intermediate feature maps never leave the SM (Sec. III-B of the
// paper: a fused layer's output is produced on chip and reused at once; Sec. IV-B: a spatial
// tile of a fused block recomputes its halo).  With one layer it is also the library's general
// stride-1 convolution kernel for narrow 3x3 layers: the input tile is read once, not once per tap.
//
// Work item = (image, output tile th x tw of the last layer).  The tile's receptive-field frame
// (th + 2 halo) x (tw + 2 halo), halo = sum of the paddings, is loaded by TMA (zero fill outside
// the image = the first layer's padding) as pixel-linear planes: row q = fy*pitch + fx holds one
// pixel's 64 channels (128 bytes, 128-byte swizzle), one plane per 64 channels.  In that layout
// tap (r, s) of a 3x3 layer is the same buffer shifted by (r-1)*pitch + (s-1) rows, so every
// layer - the first included - feeds the tensor cores straight from the resident tile through a
// shifted shared-memory descriptor: no im2col, no per-tap reload.  A layer's M dimension is the
// linear range of frame positions it must produce (wrap-around columns are computed and
// ignored), cut into 128-row blocks.  Behind the group's last 3x3 layer no halo is needed any
// more: that layer's epilogue writes the tile's own pixels densely (row = ty*tw + tx), the 1x1
// layers after it work on exactly th*tw rows, and the group's output tile leaves as whole TMA
// boxes.  A first layer that is 1x1 streams its input planes through a small ring instead of
// holding the whole frame (each plane is used once per pass).
//
// Tensor memory is split between the inner layers (columns 0..255) and the group's last layer
// (256..511), each half double-buffered, and the epilogue warps are split the same way: group A
// (warps 0-7) turns inner accumulators into the next layer's operand tile in shared memory
// (bias, activation, fp16 rounding, zero outside the image: the next layer's padding), group B
// (warps 8-15) drains the last layer (bias, residual, activation, rounding) into a swizzled
// staging tile that a store warp sends off with TMA stores; a residual tile is fetched by that
// warp with TMA loads straight into the staging buffer ahead of time and added in place.  So the
// last layer's epilogue - the longest single step of a bottleneck-shaped group - overlaps the
// next tile's first layers on the tensor cores.  Shared-memory hazards between tiles need no
// extra barriers: the tensor core executes its instructions in order, so an epilogue that was
// released by a later commit can never overwrite an operand an earlier instruction still reads.
// Pooled groups stage the whole tile and reduce 2x2 windows on the way out; tiles too large for a
// staging buffer fall back to direct 16-byte stores.
//
// Warps: 0-7 epilogue A, 8-15 epilogue B, 16 UMMA issuer (the whole warp walks the loops, one
// elected lane issues), 17-20 weight producers (a ring stage belongs to one of them), 21 input
// producer (one lane per plane of a round), 22 store warp.  Measured on B200: one TMA instruction
// keeps its issuing thread busy for about 0.28 us whatever the box size, and copies issued by
// different threads overlap: hence several producer threads and boxes of several taps / K chunks.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "internal.h"
#include "ptx.cuh"

namespace dlf {

namespace {

constexpr int kEpiWarps = 8;                   // per group
constexpr int kMmaWarp = 2 * kEpiWarps;        // warp 16: UMMA issuer, owns the TMEM allocation
constexpr int kWeightWarp0 = kMmaWarp + 1;     // warps 17..20
constexpr int kWeightWarps = 4;
constexpr int kInputWarp = kWeightWarp0 + kWeightWarps;  // warp 21
constexpr int kStoreWarp = kInputWarp + 1;               // warp 22
constexpr int kThreads = 32 * (kStoreWarp + 1);
constexpr int kWeightOpBytes = 16 * 1024;      // target size of one weight TMA box
constexpr int kMaxSmem = 232448 - 2048;        // dynamic part: the 227 KB per-CTA limit minus the static barriers and layer table
constexpr int kMaxBias = 4096;                 // floats of bias staged in shared memory (all layers)
constexpr int kMaxInSlots = 16;
constexpr int kMaxStages = 8;

enum OutMode { OUT_DIRECT = 0, OUT_STAGE = 1, OUT_POOL = 2 };

struct ChainLayerP {
    int cin, cout, k, pad, act;
    int kchunks, ksteps_last;  // 64-channel K chunks; 16-channel steps in the last one
    int qs, range, nb;         // first row produced, rows produced, 128-row blocks (in the layer's own row layout)
    int n_pad;                 // cout rounded up to 16
    int n_chunks, chunk_n;     // channel chunks of chunk_n (the last one may be smaller)
    int slot, per_pass, bgroups;  // TMEM columns per block, blocks per pass, passes per channel chunk
    int tg, kg, w_rank4;       // taps and K chunks per weight box; 4-d weight view (cin % 64 == 0)
    int w_off;                 // resident weights: byte offset of this layer's slabs, ordered [chunk][K chunk][tap][row]
    int col0, half_cols;       // TMEM region of this layer: first column, columns of one half
    int in_dense, out_dense;   // rows are tile pixels (ty*tw + tx) instead of frame positions: of the layer itself / of what it writes
    int bias_off;
    const float* bias;
};

struct ChainParams {
    CUtensorMap tmx, tmy, tmr;
    CUtensorMap tmw[kMaxChain];
    ChainLayerP L[kMaxChain];
    int n_layers;
    int N, H, W;
    int th, tw, halo, pitch, rows;  // frame geometry
    int tiles_h, tiles_w, n_tiles;
    int in_planes, in_group, in_slots, in_ring, in_slot_bytes, in_off;
    int act_off[2], act_plane_bytes[2];
    int out_mode, out_dense, out_box_rows;   // box rows of the output / residual maps: th (dense tile) or 1 (one frame row)
    int stg_off, stg_bufs, stg_buf_bytes, stg_plane_bytes, stg_base8;
    int ring_off, stages, stage_bytes, w_producers;   // stages == 0: every layer's weights stay resident in shared memory
    int bias_off, bias_floats;
    int pool;
    int cout_last;
    const __half* res;
    __half* out;
    int* status;
};

__device__ __forceinline__ void epi_bar_sync(int id) { asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(32 * kEpiWarps) : "memory"); }

__device__ __forceinline__ int chunk_cols(const ChainLayerP& L, int c) {
    return min(L.chunk_n, L.n_pad - c * L.chunk_n);
}

// Where a row of a layer lies: tile coordinates, image coordinates.
struct RowPos {
    int ty, tx, gy, gx;
    bool in_tile, in_img;
};
__device__ __forceinline__ RowPos row_pos(const ChainParams& p, bool dense, int q, int gy0, int gx0) {
    RowPos r;
    if (dense) {
        r.ty = q / p.tw;
        r.tx = q - r.ty * p.tw;
        r.in_tile = q < p.th * p.tw;
    } else {
        const int fy = q / p.pitch, fx = q - fy * p.pitch;
        r.ty = fy - p.halo;
        r.tx = fx - p.halo;
        r.in_tile = r.ty >= 0 && r.ty < p.th && r.tx >= 0 && r.tx < p.tw;
    }
    r.gy = gy0 + r.ty;
    r.gx = gx0 + r.tx;
    r.in_img = r.gy >= 0 && r.gy < p.H && r.gx >= 0 && r.gx < p.W;
    return r;
}
// Row of tile pixel (ty, tx) in the last layer's row layout.
__device__ __forceinline__ int out_row(const ChainParams& p, int ty, int tx) {
    return p.out_dense ? ty * p.tw + tx : (ty + p.halo) * p.pitch + p.halo + tx;
}

struct EpiCtx {
    int row, half;            // TMEM lane of this thread; which alternating 32-column chunks it takes
    uint32_t tmem_lane, tmem_col;
    int gy0, gx0, n;          // image coordinates of the tile's first pixel, image index
    int b0, nblk, ncols, ch0; // blocks of this pass, columns and first channel of this chunk
    uint8_t* obuf;            // buffer written (operand tile / staging tile), its plane stride
    int oplane;
    const float* bl;
    __half2 act_lo, act_hi;   // applied to rounded pairs
};

// Bias, activation (a clamp of the rounded pair, which keeps the loop free of branches), rounding of 8 channels.
__device__ __forceinline__ uint4 finish8(const float* v, const float* bias, const EpiCtx& cx) {
    const float4 b0 = *reinterpret_cast<const float4*>(bias);
    const float4 b1 = *reinterpret_cast<const float4*>(bias + 4);
    uint4 o;
    o.x = pack_half2_clamp(v[0] + b0.x, v[1] + b0.y, cx.act_lo, cx.act_hi);
    o.y = pack_half2_clamp(v[2] + b0.z, v[3] + b0.w, cx.act_lo, cx.act_hi);
    o.z = pack_half2_clamp(v[4] + b1.x, v[5] + b1.y, cx.act_lo, cx.act_hi);
    o.w = pack_half2_clamp(v[6] + b1.z, v[7] + b1.w, cx.act_lo, cx.act_hi);
    return o;
}
__device__ __forceinline__ uint4 finish8_res(const float* v, const float* bias, const uint4& rv, const EpiCtx& cx) {
    const float4 b0 = *reinterpret_cast<const float4*>(bias);
    const float4 b1 = *reinterpret_cast<const float4*>(bias + 4);
    const __half2* rh = reinterpret_cast<const __half2*>(&rv);
    const float2 r0 = __half22float2(rh[0]), r1 = __half22float2(rh[1]), r2 = __half22float2(rh[2]), r3 = __half22float2(rh[3]);
    uint4 o;
    o.x = pack_half2_clamp(v[0] + b0.x + r0.x, v[1] + b0.y + r0.y, cx.act_lo, cx.act_hi);
    o.y = pack_half2_clamp(v[2] + b0.z + r1.x, v[3] + b0.w + r1.y, cx.act_lo, cx.act_hi);
    o.z = pack_half2_clamp(v[4] + b1.x + r2.x, v[5] + b1.y + r2.y, cx.act_lo, cx.act_hi);
    o.w = pack_half2_clamp(v[6] + b1.z + r3.x, v[7] + b1.w + r3.y, cx.act_lo, cx.act_hi);
    return o;
}
// Address of 8 channels (group g8 of the buffer's channels) of row `row` in a swizzled plane buffer.
__device__ __forceinline__ uint4* tile_ptr(uint8_t* buf, int plane_bytes, int row, int g8) {
    return reinterpret_cast<uint4*>(buf + static_cast<size_t>(g8 >> 3) * plane_bytes + static_cast<size_t>(row) * 128 +
                                    (((g8 & 7) ^ (row & 7)) << 4));
}

// Drains one pass of an inner layer into the next layer's operand tile (zero outside the image).
__device__ __forceinline__ void epi_inner(const ChainParams& p, const ChainLayerP& L, const EpiCtx& cx) {
#pragma unroll 1
    for (int b = 0; b < cx.nblk; b++) {
        const int q = L.qs + (cx.b0 + b) * 128 + cx.row;
        const RowPos r = row_pos(p, L.in_dense != 0, q, cx.gy0, cx.gx0);
        bool live = q < L.qs + L.range;
        int wrow = q;
        if (L.out_dense && !L.in_dense) {   // the group's last 3x3 layer: keep the tile's own pixels, densely
            live = live && r.in_tile;
            wrow = r.ty * p.tw + r.tx;
        }
        const uint32_t taddr = cx.tmem_lane + cx.tmem_col + b * L.slot;
#pragma unroll 1
        for (int cc = cx.half * 32; cc < cx.ncols; cc += 64) {
            float v[32];
            __syncwarp();  // the aligned TMEM loads need the whole warp converged
            const int nc = min(32, cx.ncols - cc);
            if (nc == 32) tmem_ld32(taddr + cc, v);
            else tmem_ld16(taddr + cc, v);
            if (!live) continue;
#pragma unroll
            for (int g = 0; g < 4; g++) {
                if (g * 8 >= nc) break;
                const int co = cx.ch0 + cc + g * 8;  // first of 8 channels
                // channels past cout (padding up to 16) carry zero weights and zero bias: act(0) = 0,
                // so the next layer's K padding stays zero
                const uint4 val = r.in_img ? finish8(v + g * 8, cx.bl + co, cx) : make_uint4(0u, 0u, 0u, 0u);
                *tile_ptr(cx.obuf, cx.oplane, wrow, co >> 3) = val;
            }
        }
    }
}

// Drains one pass of the group's last layer.  MODE OUT_DIRECT: 16-byte global stores (residual by global loads);
// OUT_STAGE: staging tile (the residual, if any, already lies there); OUT_POOL: staging tile of the whole frame.
template <int MODE>
__device__ __forceinline__ void epi_last(const ChainParams& p, const ChainLayerP& L, const EpiCtx& cx) {
    const bool has_res = p.res != nullptr;
#pragma unroll 1
    for (int b = 0; b < cx.nblk; b++) {
        const int q = L.qs + (cx.b0 + b) * 128 + cx.row;
        const RowPos r = row_pos(p, L.in_dense != 0, q, cx.gy0, cx.gx0);
        const bool live = q < L.qs + L.range && (MODE == OUT_POOL || (r.in_tile && r.in_img));
        const long long gpix = (static_cast<long long>(cx.n) * p.H + r.gy) * p.W + r.gx;
        const int srow = q - p.stg_base8;
        const uint32_t taddr = cx.tmem_lane + cx.tmem_col + b * L.slot;
#pragma unroll 1
        for (int cc = cx.half * 32; cc < cx.ncols; cc += 64) {
            float v[32];
            __syncwarp();
            const int nc = min(32, cx.ncols - cc);
            if (nc == 32) tmem_ld32(taddr + cc, v);
            else tmem_ld16(taddr + cc, v);
            if (!live) continue;
#pragma unroll
            for (int g = 0; g < 4; g++) {
                if (g * 8 >= nc) break;
                const int co = cx.ch0 + cc + g * 8;
                if (MODE == OUT_STAGE) {
                    uint4* sp = tile_ptr(cx.obuf, cx.oplane, srow, (cc >> 3) + g);
                    *sp = has_res ? finish8_res(v + g * 8, cx.bl + co, *sp, cx) : finish8(v + g * 8, cx.bl + co, cx);
                } else {
                    uint4 val;
                    if (has_res && co < L.cout && r.in_tile && r.in_img)
                        val = finish8_res(v + g * 8, cx.bl + co, __ldg(reinterpret_cast<const uint4*>(p.res + gpix * L.cout + co)), cx);
                    else
                        val = finish8(v + g * 8, cx.bl + co, cx);
                    if (MODE == OUT_POOL) *tile_ptr(cx.obuf, cx.oplane, srow, co >> 3) = val;
                    else if (co < L.cout) *reinterpret_cast<uint4*>(p.out + gpix * L.cout + co) = val;
                }
            }
        }
    }
}

// The UMMAs of one pass whose operands are all in shared memory already (resident weights; an operand tile of the group,
// or a resident input frame): for every 64-channel chunk, every tap, every block of the pass, four K = 16 steps.  The
// issuing warp is bound by its own instruction stream (measured: about 4 cycles per instruction, and a pass of 36 UMMAs
// cost it 3000 instructions in the general loop below), so this path is kept to a few instructions per UMMA: 32-bit
// descriptor words, the tap loop unrolled at compile time, nothing but adds inside.
//   a16 / b16: low descriptor words of tap (0, 0), chunk 0, block 0 / of the first weight slab
template <int K>
__device__ __forceinline__ void issue_pass_resident(uint32_t d0, uint32_t slot_cols, int nblk, uint32_t a16, uint32_t a_chunk16, uint32_t b16,
                                                    uint32_t w_tap16, uint32_t idesc, int kchunks, int ksteps_last, int pitch) {
#pragma unroll 1
    for (int kc = 0; kc < kchunks; kc++, a16 += a_chunk16) {
        const bool whole = kc + 1 < kchunks || ksteps_last == 4;
#pragma unroll
        for (int r = 0; r < K; r++) {
#pragma unroll
            for (int sx = 0; sx < K; sx++) {
                uint32_t a = a16 + static_cast<uint32_t>((r * pitch + sx) * 8), d = d0;
                const uint32_t acc = (kc | r | sx) != 0;
#pragma unroll 1
                for (int blk = 0; blk < nblk; blk++, a += (128 * 128) >> 4, d += slot_cols) {
                    if (elect_one()) {
                        if (whole) {
                            umma_f16_x4(d, a, b16, idesc, acc);
                        } else {
                            umma_f16_lo(d, a, kDescHiSw128, b16, idesc, acc);
                            if (ksteps_last > 1) umma_f16_lo(d, a + 2, kDescHiSw128, b16 + 2, idesc, 1);
                            if (ksteps_last > 2) umma_f16_lo(d, a + 4, kDescHiSw128, b16 + 4, idesc, 1);
                        }
                    }
                }
                b16 += w_tap16;
            }
        }
    }
}

template <int OUT_MODE>
__global__ void __launch_bounds__(kThreads, 1) chain_tc_kernel(const __grid_constant__ ChainParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t wfull_bar[kMaxStages], wempty_bar[kMaxStages], in_full_bar[kMaxInSlots], in_empty_bar[kMaxInSlots];
    __shared__ uint64_t acc_full_bar[4], acc_empty_bar[4];  // [region * 2 + half]; region 0 = inner layers, 1 = last layer
    __shared__ uint64_t act_ready_bar, stg_full_bar[2], stg_free_bar[2], wres_bar[kMaxChain];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    // The layers' parameters, copied out of the kernel's parameter block: every role walks the layers of every tile, and
    // a dynamically indexed read of the parameter block cost the issuing warp about 700 cycles per layer (measured).
    __shared__ __align__(16) ChainLayerP Ls[kMaxChain];

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sbase = smem_raw + (base - smem_u32(smem_raw));
    float* bias_s = reinterpret_cast<float*>(sbase + p.bias_off);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = &abort_s;
    const int nl = p.n_layers;
    {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(&p.L[0]);
        uint32_t* dst = reinterpret_cast<uint32_t*>(&Ls[0]);
        const int words = nl * static_cast<int>(sizeof(ChainLayerP) / 4);
#pragma unroll 1
        for (int i = threadIdx.x; i < words; i += kThreads) dst[i] = src[i];
    }
    const ChainLayerP& LL = Ls[nl - 1];

    if (threadIdx.x == 0) {
        DLF_TRACE_POINT(p.status, 24);
        abort_s = 0;
#pragma unroll 1
        for (int i = 0; i < p.stages; i++) {
            mbar_init(&wfull_bar[i], 1);
            mbar_init(&wempty_bar[i], 1);
        }
#pragma unroll 1
        for (int i = 0; i < p.in_slots; i++) {
            mbar_init(&in_full_bar[i], 1);
            mbar_init(&in_empty_bar[i], 1);
        }
#pragma unroll 1
        for (int i = 0; i < 4; i++) {
            mbar_init(&acc_full_bar[i], 1);
            mbar_init(&acc_empty_bar[i], kEpiWarps);
        }
        mbar_init(&act_ready_bar, kEpiWarps);
#pragma unroll 1
        for (int i = 0; i < kMaxChain; i++) mbar_init(&wres_bar[i], kWeightWarps);
#pragma unroll 1
        for (int i = 0; i < 2; i++) {
            mbar_init(&stg_full_bar[i], kEpiWarps);
            mbar_init(&stg_free_bar[i], 1);
        }
        fence_barrier_init();
        tma_prefetch_desc(&p.tmx);
        if (OUT_MODE == OUT_STAGE) {
            tma_prefetch_desc(&p.tmy);
            if (p.res != nullptr) tma_prefetch_desc(&p.tmr);
        }
    }
    if (warp == kMmaWarp) {
        tmem_alloc(&tmem_base_s, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();
    // the set-up above overlapped the previous kernel; from here on its outputs are read - except by the
    // weight producers, which only read constants and may run ahead
    if (warp < kWeightWarp0 || warp >= kInputWarp) pdl_wait();
    // All 512 columns are allocated, so the allocation starts at lane 0, column 0: the literal keeps every tensor-memory
    // address a compile-time-uniform value (an address loaded from shared memory is a per-thread value to the compiler
    // and costs a move into a uniform register at every UMMA).  Checked once; a surprise is reported, not ignored.
    constexpr uint32_t tmem_base = 0;
    if (threadIdx.x == 0 && tmem_base_s != 0u) {
        abort_s = 1;
        atomicCAS(p.status, 0, 0xb00 | (blockIdx.x << 12));
    }
    const int ring_rounds = p.in_slots / p.in_group;     // producer rounds the input slots hold
    const int rounds_per_pass = p.in_planes / p.in_group;
    const int passes0 = p.L[0].n_chunks * p.L[0].bgroups;   // (statically indexed: read before the copy above is visible)

    if (warp == kInputWarp) {
        // ---- input producer: a round = in_group planes, one lane each; a lane owns its slots ---------------
        if (lane < p.in_group) {
            const uint32_t plane_bytes = static_cast<uint32_t>(p.rows * p.pitch) * 128u;
            const int rounds_per_tile = p.in_ring ? passes0 * rounds_per_pass : 1;
            int rd = 0;           // round within the slots
            uint32_t ph = 0;      // phase of the slots' barriers
            bool ok = true;
#pragma unroll 1
            for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x) {
                const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h, n = t / (p.tiles_w * p.tiles_h);
                int plane = lane;
#pragma unroll 1
                for (int rr = 0; rr < rounds_per_tile; rr++) {
                    const int slot = rd * p.in_group + lane;
                    ok = mbar_wait(&in_empty_bar[slot], ph ^ 1u, abort_flag, p.status, 0x100 | (blockIdx.x << 12));
                    if (!ok) break;
                    mbar_expect_tx(&in_full_bar[slot], plane_bytes);
                    tma_load_4d(sbase + p.in_off + static_cast<size_t>(slot) * p.in_slot_bytes, &p.tmx, &in_full_bar[slot], plane * 64,
                                txi * p.tw - p.halo, tyi * p.th - p.halo, n);
                    plane += p.in_group;
                    if (plane >= p.in_planes) plane = lane;
                    if (++rd == ring_rounds) { rd = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp >= kWeightWarp0 && warp < kWeightWarp0 + kWeightWarps) {
        // ---- weight producers: one box of tg taps x kg K chunks x [chunk_n][64] per ring stage ------
        const int role = warp - kWeightWarp0;
        if (lane == 0 && p.stages == 0) {
            // resident weights: every layer's slabs are loaded once, the boxes dealt out to the four producers in turn
#pragma unroll 1
            for (int l = 0; l < nl; l++) {
                const ChainLayerP& L = Ls[l];
                const int taps = L.k * L.k, tg = L.tg, kg = L.kg, kchunks = L.kchunks, rank4 = L.w_rank4;
                const uint32_t bytes = static_cast<uint32_t>(tg * kg * L.chunk_n) * 128u;
                const int n_boxes = L.n_chunks * (taps / tg) * (kchunks / kg);
                mbar_expect_tx(&wres_bar[l], static_cast<uint32_t>((n_boxes - role + kWeightWarps - 1) / kWeightWarps) * bytes);
                // Every CTA wants the same slabs at the same moment: each starts its round at another box, so that the
                // requests of the 148 CTAs spread over the L2 slices instead of queueing on the same lines.
                const int first = (static_cast<int>(blockIdx.x) * kWeightWarps) % n_boxes;
                int turn = 0, box = 0;
#pragma unroll 1
                for (int c = 0; c < L.n_chunks; c++)
#pragma unroll 1
                    for (int t0 = 0; t0 < taps; t0 += tg)
#pragma unroll 1
                        for (int g0 = 0; g0 < kchunks; g0 += kg, box++) {
                            if (turn == role && box >= first) {
                                if (l == 0 && role == 0 && box == first) DLF_TRACE_POINT(p.status, 25);
                                uint8_t* dst = sbase + p.ring_off + L.w_off + static_cast<size_t>((c * kchunks + g0) * taps + t0) * L.chunk_n * 128;
                                if (rank4) tma_load_4d(dst, &p.tmw[l], &wres_bar[l], 0, c * L.chunk_n, t0, g0);
                                else tma_load_3d(dst, &p.tmw[l], &wres_bar[l], g0 * 64, c * L.chunk_n, t0);
                            }
                            if (++turn == kWeightWarps) turn = 0;
                        }
                turn = 0, box = 0;   // ... and the boxes before its starting point afterwards
#pragma unroll 1
                for (int c = 0; c < L.n_chunks && box < first; c++)
#pragma unroll 1
                    for (int t0 = 0; t0 < taps && box < first; t0 += tg)
#pragma unroll 1
                        for (int g0 = 0; g0 < kchunks && box < first; g0 += kg, box++) {
                            if (turn == role) {
                                uint8_t* dst = sbase + p.ring_off + L.w_off + static_cast<size_t>((c * kchunks + g0) * taps + t0) * L.chunk_n * 128;
                                if (rank4) tma_load_4d(dst, &p.tmw[l], &wres_bar[l], 0, c * L.chunk_n, t0, g0);
                                else tma_load_3d(dst, &p.tmw[l], &wres_bar[l], g0 * 64, c * L.chunk_n, t0);
                            }
                            if (++turn == kWeightWarps) turn = 0;
                        }
            }
        } else if (lane == 0 && role < p.w_producers) {
            int st = 0, turn = 0;   // ring stage of the next box; whose turn it is (a stage belongs to one producer:
            uint32_t ph = 0;        // the stage count is a multiple of the producers)
            bool ok = true;
#pragma unroll 1
            for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x) {
#pragma unroll 1
                for (int l = 0; l < nl && ok; l++) {
                    const ChainLayerP& L = Ls[l];
                    const uint32_t bytes = static_cast<uint32_t>(L.tg * L.kg * L.chunk_n) * 128u;  // the whole box
                    const int taps = L.k * L.k, tg = L.tg, kg = L.kg, kchunks = L.kchunks, rank4 = L.w_rank4;
#pragma unroll 1
                    for (int c = 0; c < L.n_chunks && ok; c++)
#pragma unroll 1
                        for (int ps = 0; ps < L.bgroups && ok; ps++)
#pragma unroll 1
                            for (int t0 = 0; t0 < taps && ok; t0 += tg)
#pragma unroll 1
                                for (int g0 = 0; g0 < kchunks; g0 += kg) {
                                    if (turn == role) {
                                        ok = mbar_wait(&wempty_bar[st], ph ^ 1u, abort_flag, p.status, 0x200 | (blockIdx.x << 12));
                                        if (!ok) break;
                                        mbar_expect_tx(&wfull_bar[st], bytes);
                                        uint8_t* dst = sbase + p.ring_off + static_cast<size_t>(st) * p.stage_bytes;
                                        if (rank4) tma_load_4d(dst, &p.tmw[l], &wfull_bar[st], 0, c * L.chunk_n, t0, g0);
                                        else tma_load_3d(dst, &p.tmw[l], &wfull_bar[st], g0 * 64, c * L.chunk_n, t0);
                                    }
                                    if (++turn == p.w_producers) turn = 0;
                                    if (++st == p.stages) { st = 0; ph ^= 1u; }
                                }
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ---- UMMA issuer: the whole warp walks the loops (warp-uniform addresses), one elected lane issues ----
        // Ring positions and phases are kept as counters: a division by a run-time value costs this single warp about a
        // hundred cycles, and the loop around a weight box issues as few as four instructions.
        const uint64_t desc0 = umma_desc_sw128(0);
        uint32_t pass_ctr[2] = {0, 0}, act_ph = 0, w_ph = 0, in_ph = 0;
        int w_st = 0, in_rd = 0, in_j = 0;   // weight stage; input round within the slots and (streamed planes) plane within the round
        const int in_group = p.in_group, in_ring = p.in_ring, pitch = p.pitch, stages = p.stages;
        const uint32_t in_base = base + p.in_off, in_slot_bytes = p.in_slot_bytes;
        bool ok = true;
        DLF_TRACE_DECL(tacc, tmark);  // cycles of CTA 0's issuer: 0 input wait, 1 layer hand-off wait, 2 accumulator wait, 3 weight wait, 4 issue
#pragma unroll 1
        for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x) {
#pragma unroll 1
            for (int l = 0; l < nl && ok; l++) {
                const ChainLayerP& L = Ls[l];
                const int region = (l == nl - 1) ? 1 : 0;
                if (l > 0) {  // group A has written all of the previous layer's tile
                    ok = mbar_wait_warp<true>(&act_ready_bar, act_ph, abort_flag, p.status, 0x400 | (blockIdx.x << 12));
                    if (!ok) break;
                    act_ph ^= 1u;
                    DLF_TRACE_ACC(tacc, 1, tmark);
                }
                const uint32_t abuf = l == 0 ? 0u : base + p.act_off[(l - 1) & 1];
                const uint32_t aplane_bytes = l == 0 ? 0u : static_cast<uint32_t>(p.act_plane_bytes[(l - 1) & 1]);
                const int k = L.k, pad = L.pad, taps = k * k, tg = L.tg, kg = L.kg, kchunks = L.kchunks, ksteps_last = L.ksteps_last;
                const int nb = L.nb, per_pass = L.per_pass, n_chunks = L.n_chunks;
                const uint32_t slot_cols = L.slot, col0 = L.col0, half_cols = L.half_cols, qs = L.qs;
                const uint32_t w_tap16 = static_cast<uint32_t>(L.chunk_n) * 8u;  // one tap's [chunk_n][64] slab, 16-byte units
                const bool w_res = stages == 0;
                if (w_res) {   // this layer's resident weights have landed (true at once from the second tile on)
                    ok = mbar_wait_warp<true>(&wres_bar[l], 0u, abort_flag, p.status, 0x600 | (blockIdx.x << 12));
                    if (!ok) break;
                    if (l == 0 && t == static_cast<int>(blockIdx.x) && lane == 0) DLF_TRACE_POINT(p.status, 26);
                    DLF_TRACE_ACC(tacc, 3, tmark);
                }
                const uint32_t w_res0 = base + p.ring_off + L.w_off;
                bool first_pass = true;
#pragma unroll 1
                for (int c = 0; c < n_chunks && ok; c++) {
                    const uint32_t idesc = umma_idesc_f16(chunk_cols(L, c));
#pragma unroll 1
                    for (int b0 = 0; b0 < nb && ok; b0 += per_pass) {
                        const int nblk = min(per_pass, nb - b0);
                        const uint32_t pc = pass_ctr[region]++;
                        const uint32_t half = pc & 1u;
                        ok = mbar_wait_warp<true>(&acc_empty_bar[region * 2 + half], ((pc >> 1) & 1u) ^ 1u, abort_flag, p.status,
                                            0x500 | (blockIdx.x << 12));
                        if (!ok) break;
                        DLF_TRACE_ACC(tacc, 2, tmark);
                        tc_fence_after_sync();
                        const uint32_t d_tmem0 = tmem_base + col0 + half * half_cols;
                        const uint32_t row0 = (qs + static_cast<uint32_t>(b0) * 128u) * 128u;
                        if (w_res && !(l == 0 && in_ring)) {
                            // ---- the lean path: every operand of the pass is in shared memory ----------------------
                            if (l == 0 && first_pass) {   // the tile's input frame has landed
#pragma unroll 1
                                for (int kc = 0; kc < kchunks && ok; kc++)
                                    ok = mbar_wait_warp<true>(&in_full_bar[in_rd * in_group + kc], in_ph, abort_flag, p.status, 0x300 | (blockIdx.x << 12));
                                if (!ok) break;
                                if (t == static_cast<int>(blockIdx.x) && lane == 0) DLF_TRACE_POINT(p.status, 27);
                                DLF_TRACE_ACC(tacc, 0, tmark);
                            }
                            const uint32_t a_base = l == 0 ? in_base + static_cast<uint32_t>(in_rd * in_group) * in_slot_bytes : abuf;
                            const uint32_t a_chunk16 = (l == 0 ? in_slot_bytes : aplane_bytes) >> 4;
                            const uint32_t a16 = umma_desc_lo(a_base + row0) - static_cast<uint32_t>(pad * (pitch + 1) * 8);
                            const uint32_t b16 = umma_desc_lo(w_res0) + static_cast<uint32_t>(c * kchunks * taps) * w_tap16;
                            if (k == 3) issue_pass_resident<3>(d_tmem0, slot_cols, nblk, a16, a_chunk16, b16, w_tap16, idesc, kchunks, ksteps_last, pitch);
                            else issue_pass_resident<1>(d_tmem0, slot_cols, nblk, a16, a_chunk16, b16, w_tap16, idesc, kchunks, ksteps_last, pitch);
                            DLF_TRACE_ACC(tacc, 4, tmark);
                            if (elect_one()) umma_commit(&acc_full_bar[region * 2 + half]);
                            __syncwarp();
                            first_pass = false;
                            continue;
                        }
                        if (w_res && l == 0 && in_ring) {
                            // ---- lean path of a 1x1 first layer whose input planes stream through the slots ----------
                            uint32_t b16 = umma_desc_lo(w_res0) + static_cast<uint32_t>(c * kchunks) * w_tap16;
#pragma unroll 1
                            for (int kc = 0; kc < kchunks && ok; kc++, b16 += w_tap16) {
                                const int in_slot = in_rd * in_group + in_j;
                                ok = mbar_wait_warp<true>(&in_full_bar[in_slot], in_ph, abort_flag, p.status, 0x300 | (blockIdx.x << 12));
                                if (!ok) break;
                                uint32_t a = umma_desc_lo(in_base + static_cast<uint32_t>(in_slot) * in_slot_bytes + row0), d = d_tmem0;
                                const bool whole = kc + 1 < kchunks || ksteps_last == 4;
#pragma unroll 1
                                for (int blk = 0; blk < nblk; blk++, a += (128 * 128) >> 4, d += slot_cols) {
                                    if (elect_one()) {
                                        if (whole) {
                                            umma_f16_x4(d, a, b16, idesc, kc != 0);
                                        } else {
                                            umma_f16_lo(d, a, kDescHiSw128, b16, idesc, kc != 0);
                                            if (ksteps_last > 1) umma_f16_lo(d, a + 2, kDescHiSw128, b16 + 2, idesc, 1);
                                            if (ksteps_last > 2) umma_f16_lo(d, a + 4, kDescHiSw128, b16 + 4, idesc, 1);
                                        }
                                    }
                                }
                                if (elect_one()) umma_commit(&in_empty_bar[in_slot]);   // the plane is free once these have read it
                                if (++in_j == in_group) { in_j = 0; if (++in_rd == ring_rounds) { in_rd = 0; in_ph ^= 1u; } }
                            }
                            if (!ok) break;
                            DLF_TRACE_ACC(tacc, 4, tmark);
                            if (elect_one()) umma_commit(&acc_full_bar[region * 2 + half]);
                            __syncwarp();
                            first_pass = false;
                            continue;
                        }
                        // ---- weights streamed through the ring: one box = tg taps x kg chunks, waited for and released as a whole ----
                        {
                            const uint32_t a_base = l == 0 ? in_base + static_cast<uint32_t>(in_rd * in_group) * in_slot_bytes : abuf;
                            const uint32_t a_chunk16 = (l == 0 ? in_slot_bytes : aplane_bytes) >> 4;
                            const uint32_t a16 = umma_desc_lo(a_base + row0) - static_cast<uint32_t>(pad * (pitch + 1) * 8);
                            const bool a_ring = l == 0 && in_ring;   // (then k == 1: the planes come through the slots one by one)
                            if (l == 0 && !in_ring && first_pass) {   // the tile's input frame has landed
#pragma unroll 1
                                for (int kc = 0; kc < kchunks && ok; kc++)
                                    ok = mbar_wait_warp<true>(&in_full_bar[in_rd * in_group + kc], in_ph, abort_flag, p.status, 0x300 | (blockIdx.x << 12));
                                if (!ok) break;
                                DLF_TRACE_ACC(tacc, 0, tmark);
                            }
                            int r0 = 0, sx0 = 0;   // kernel row / column of tap t0
#pragma unroll 1
                            for (int t0 = 0; t0 < taps && ok; t0 += tg) {
#pragma unroll 1
                                for (int g0 = 0; g0 < kchunks && ok; g0 += kg) {
                                    ok = mbar_wait_warp<true>(&wfull_bar[w_st], w_ph, abort_flag, p.status, 0x600 | (blockIdx.x << 12));
                                    if (!ok) break;
                                    DLF_TRACE_ACC(tacc, 3, tmark);
                                    uint32_t b16 = umma_desc_lo(base + p.ring_off + w_st * p.stage_bytes);
                                    const int g_end = min(kg, kchunks - g0);
#pragma unroll 1
                                    for (int g = 0; g < g_end && ok; g++) {
                                        const int kc = g0 + g;
                                        const bool whole = kc + 1 < kchunks || ksteps_last == 4;
                                        uint32_t a_kc;
                                        int in_slot = 0;
                                        if (a_ring) {
                                            in_slot = in_rd * in_group + in_j;
                                            ok = mbar_wait_warp<true>(&in_full_bar[in_slot], in_ph, abort_flag, p.status, 0x300 | (blockIdx.x << 12));
                                            if (!ok) break;
                                            a_kc = umma_desc_lo(in_base + static_cast<uint32_t>(in_slot) * in_slot_bytes + row0);
                                        } else {
                                            a_kc = a16 + static_cast<uint32_t>(kc) * a_chunk16;
                                        }
                                        uint32_t shift16 = static_cast<uint32_t>((r0 * pitch + sx0) * 8);
                                        int sx = sx0;
                                        uint32_t acc = (r0 | sx0 | kc) != 0;
#pragma unroll 1
                                        for (int tt = 0; tt < tg; tt++, b16 += w_tap16) {
                                            uint32_t a = a_kc + shift16, d = d_tmem0;
#pragma unroll 1
                                            for (int blk = 0; blk < nblk; blk++, a += (128 * 128) >> 4, d += slot_cols) {
                                                if (elect_one()) {
                                                    if (whole) {
                                                        umma_f16_x4(d, a, b16, idesc, acc);
                                                    } else {
                                                        umma_f16_lo(d, a, kDescHiSw128, b16, idesc, acc);
                                                        if (ksteps_last > 1) umma_f16_lo(d, a + 2, kDescHiSw128, b16 + 2, idesc, 1);
                                                        if (ksteps_last > 2) umma_f16_lo(d, a + 4, kDescHiSw128, b16 + 4, idesc, 1);
                                                    }
                                                }
                                            }
                                            acc = 1;
                                            shift16 += 8;
                                            if (++sx == k) { sx = 0; shift16 += static_cast<uint32_t>((pitch - k) * 8); }
                                        }
                                        if (a_ring) {   // the plane is free once these have read it
                                            if (elect_one()) umma_commit(&in_empty_bar[in_slot]);
                                            if (++in_j == in_group) { in_j = 0; if (++in_rd == ring_rounds) { in_rd = 0; in_ph ^= 1u; } }
                                        }
                                    }
                                    if (!ok) break;
                                    if (elect_one()) umma_commit(&wempty_bar[w_st]);
                                    __syncwarp();
                                    if (++w_st == stages) { w_st = 0; w_ph ^= 1u; }
                                    DLF_TRACE_ACC(tacc, 4, tmark);
                                }
                                sx0 += tg;
                                while (sx0 >= k) { sx0 -= k; r0++; }
                            }
                        }
                        if (ok && elect_one()) umma_commit(&acc_full_bar[region * 2 + half]);
                        __syncwarp();
                        first_pass = false;
                    }
                }
                // a resident input frame is read by the first layer only
                if (l == 0 && !in_ring) {
                    if (ok && elect_one())
#pragma unroll 1
                        for (int kc = 0; kc < p.in_planes; kc++) umma_commit(&in_empty_bar[in_rd * in_group + kc]);
                    __syncwarp();
                    if (++in_rd == ring_rounds) { in_rd = 0; in_ph ^= 1u; }
                }
            }
        }
        if (lane == 0) DLF_TRACE_FLUSH_AT(p.status, tacc, 0);
    } else if (warp < kEpiWarps) {
        // ---- epilogue group A: inner layers -> next operand tile ---------------------------------------------
        const int et = threadIdx.x;  // 0 .. 32*kEpiWarps-1
        // biases staged by the epilogue warps alone, behind the CTA-wide barrier: the producers' first copies do not
        // wait for these loads
#pragma unroll 1
        for (int l = 0; l < nl - 1; l++) {
            const ChainLayerP& L = Ls[l];
#pragma unroll 1
            for (int i = et; i < L.n_pad; i += 32 * kEpiWarps) bias_s[L.bias_off + i] = i < L.cout ? __ldg(L.bias + i) : 0.0f;
        }
        epi_bar_sync(1);
        EpiCtx cx;
        cx.row = (warp & 3) * 32 + lane;
        cx.half = warp >> 2;
        cx.tmem_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        uint32_t pass_i = 0;
        bool ok = nl > 1;
        DLF_TRACE_DECL(aacc, amark);  // cycles of CTA 0's first group-A thread: 0 accumulator wait, 1 drain, 2 fences and arrivals
#pragma unroll 1
        for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x) {
            const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h;
            cx.gy0 = tyi * p.th;
            cx.gx0 = txi * p.tw;
            cx.n = t / (p.tiles_w * p.tiles_h);
#pragma unroll 1
            for (int l = 0; l < nl - 1 && ok; l++) {
                const ChainLayerP& L = Ls[l];
                cx.obuf = sbase + p.act_off[l & 1];
                cx.oplane = p.act_plane_bytes[l & 1];
                cx.bl = bias_s + L.bias_off;
                cx.act_lo = __float2half2_rn(L.act >= 1 ? 0.0f : -INFINITY);
                cx.act_hi = __float2half2_rn(L.act == 2 ? 6.0f : INFINITY);
#pragma unroll 1
                for (int c = 0; c < L.n_chunks && ok; c++) {
                    cx.ncols = chunk_cols(L, c);
                    cx.ch0 = c * L.chunk_n;
#pragma unroll 1
                    for (int b0 = 0; b0 < L.nb && ok; b0 += L.per_pass, pass_i++) {
                        const uint32_t half = pass_i & 1u;
                        ok = mbar_wait<true>(&acc_full_bar[half], (pass_i >> 1) & 1u, abort_flag, p.status, 0x700 | (blockIdx.x << 12));
                        if (!ok) break;
                        DLF_TRACE_ACC(aacc, 0, amark);
                        tc_fence_after_sync();
                        cx.b0 = b0;
                        cx.nblk = min(L.per_pass, L.nb - b0);
                        cx.tmem_col = L.col0 + half * L.half_cols;
                        epi_inner(p, L, cx);
                        DLF_TRACE_ACC(aacc, 1, amark);
                        fence_proxy_async_smem();  // UMMA reads these rows through the async proxy
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&acc_empty_bar[half]);
                    }
                }
                if (ok && lane == 0) mbar_arrive(&act_ready_bar);
                DLF_TRACE_ACC(aacc, 2, amark);
            }
        }
        if (et == 0) DLF_TRACE_FLUSH_AT(p.status, aacc, 16);
    } else if (warp < 2 * kEpiWarps) {
        // ---- epilogue group B: the group's last layer --------------------------------------------------------------
        const int et = threadIdx.x - 32 * kEpiWarps;
        const int wb = warp - kEpiWarps;
#pragma unroll 1
        for (int i = et; i < LL.n_pad; i += 32 * kEpiWarps) bias_s[LL.bias_off + i] = i < LL.cout ? __ldg(LL.bias + i) : 0.0f;
        epi_bar_sync(2);
        EpiCtx cx;
        cx.row = (wb & 3) * 32 + lane;
        cx.half = wb >> 2;
        cx.tmem_lane = tmem_base + (static_cast<uint32_t>((wb & 3) * 32) << 16);
        cx.bl = bias_s + LL.bias_off;
        cx.act_lo = __float2half2_rn(LL.act >= 1 ? 0.0f : -INFINITY);
        cx.act_hi = __float2half2_rn(LL.act == 2 ? 6.0f : INFINITY);
        cx.oplane = p.stg_plane_bytes;
        uint32_t pass_i = 0, use_i = 0;
        bool ok = true;
        DLF_TRACE_DECL(eacc, emark);  // cycles of CTA 0's first group-B thread: 0 staging wait, 1 accumulator wait, 2 drain, 3 pooled copy-out
#pragma unroll 1
        for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x) {
            const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h, n = t / (p.tiles_w * p.tiles_h);
            cx.gy0 = tyi * p.th;
            cx.gx0 = txi * p.tw;
            cx.n = n;
#pragma unroll 1
            for (int c = 0; c < LL.n_chunks && ok; c++) {
                cx.ncols = chunk_cols(LL, c);
                cx.ch0 = c * LL.chunk_n;
                uint32_t sb = 0;
                if (OUT_MODE == OUT_STAGE) {   // one staging buffer per channel chunk (all of its blocks are one pass)
                    sb = use_i % p.stg_bufs;
                    const uint32_t ph = (use_i / p.stg_bufs) & 1u;
                    // free again (first uses pass at once) / holds this chunk's residual
                    ok = mbar_wait(&stg_free_bar[sb], p.res != nullptr ? ph : ph ^ 1u, abort_flag, p.status, 0x800 | (blockIdx.x << 12));
                    if (!ok) break;
                    cx.obuf = sbase + p.stg_off + sb * p.stg_buf_bytes;
                    use_i++;
                } else {
                    cx.obuf = sbase + p.stg_off;
                }
                DLF_TRACE_ACC(eacc, 0, emark);
#pragma unroll 1
                for (int b0 = 0; b0 < LL.nb && ok; b0 += LL.per_pass, pass_i++) {
                    const uint32_t half = pass_i & 1u;
                    ok = mbar_wait(&acc_full_bar[2 + half], (pass_i >> 1) & 1u, abort_flag, p.status, 0x900 | (blockIdx.x << 12));
                    if (!ok) break;
                    DLF_TRACE_ACC(eacc, 1, emark);
                    tc_fence_after_sync();
                    cx.b0 = b0;
                    cx.nblk = min(LL.per_pass, LL.nb - b0);
                    cx.tmem_col = LL.col0 + half * LL.half_cols;
                    epi_last<OUT_MODE>(p, LL, cx);
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty_bar[2 + half]);
                    DLF_TRACE_ACC(eacc, 2, emark);
                }
                if (ok && OUT_MODE == OUT_STAGE) {
                    fence_proxy_async_smem();  // the staging tile is read by the TMA unit
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&stg_full_bar[sb]);
                }
            }
            if (!ok) break;
            if (OUT_MODE == OUT_POOL) {
                // ---- pooled copy-out from the staging tile (coalesced 16-byte stores) -----------------
                epi_bar_sync(2);
                const uint8_t* obuf = sbase + p.stg_off;
                const int c8n = p.cout_last / 8;
                const int oth = p.th / 2, otw = p.tw / 2;
                const int Ho = p.H / 2, Wo = p.W / 2;
                const int total = oth * otw * c8n;
#pragma unroll 1
                for (int i = et; i < total; i += 32 * kEpiWarps) {
                    const int g8 = i % c8n;
                    const int ox = (i / c8n) % otw, oy = i / (c8n * otw);
                    const int gy = tyi * oth + oy, gx = txi * otw + ox;
                    if (gy >= Ho || gx >= Wo) continue;
                    uint4 best = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int wq = 0; wq < 4; wq++) {
                        const int q = out_row(p, oy * 2 + (wq >> 1), ox * 2 + (wq & 1)) - p.stg_base8;
                        const uint4 vv = *reinterpret_cast<const uint4*>(obuf + static_cast<size_t>(g8 >> 3) * p.stg_plane_bytes +
                                                                         static_cast<size_t>(q) * 128 + (((g8 & 7) ^ (q & 7)) << 4));
                        if (wq == 0) {
                            best = vv;
                        } else {
                            __half2* bh = reinterpret_cast<__half2*>(&best);
                            const __half2* vh = reinterpret_cast<const __half2*>(&vv);
#pragma unroll
                            for (int e = 0; e < 4; e++) bh[e] = __hmax2(bh[e], vh[e]);
                        }
                    }
                    *reinterpret_cast<uint4*>(p.out + ((static_cast<long long>(n) * Ho + gy) * Wo + gx) * p.cout_last + g8 * 8) = best;
                }
                epi_bar_sync(2);
                DLF_TRACE_ACC(eacc, 3, emark);
            }
        }
        if (et == 0) DLF_TRACE_FLUSH_AT(p.status, eacc, 8);
    } else if (warp == kStoreWarp) {
        // ---- store warp: staged chunks out by TMA stores, residual chunks in by TMA loads ---------------------------
        // One lane per box (a 64-channel plane of the dense tile, or of one frame row): a thread's bulk copies run one
        // after the other, the copies of different lanes side by side.
        if (OUT_MODE == OUT_STAGE) {
            const bool has_res = p.res != nullptr;
            const int n_chunks = LL.n_chunks;
            // boxes of chunk c of tile t: planes x (1 box for a dense tile | one per tile row inside the image)
            auto boxes_of = [&](int t, int c, int* rows_in) {
                const int tyi = (t / p.tiles_w) % p.tiles_h;
                const int planes = (chunk_cols(LL, c) + 63) >> 6;
                *rows_in = p.out_dense ? 1 : min(p.th, p.H - tyi * p.th);
                return planes * *rows_in;
            };
            auto box_args = [&](int t, int c, int it, int rows_in, uint32_t sb, uint8_t** smem, int* c0, int* c1, int* c2, int* c3) {
                const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h, n = t / (p.tiles_w * p.tiles_h);
                const int pl = it / rows_in, ty = it - pl * rows_in;
                const int srow = p.out_dense ? 0 : out_row(p, ty, 0) - p.stg_base8;
                *smem = sbase + p.stg_off + sb * p.stg_buf_bytes + static_cast<size_t>(pl) * p.stg_plane_bytes + static_cast<size_t>(srow) * 128;
                *c0 = c * LL.chunk_n + pl * 64;
                *c1 = txi * p.tw;
                *c2 = tyi * p.th + ty;
                *c3 = n;
            };
            auto fetch_residual = [&](uint32_t u) {   // the u-th (tile, chunk) of this CTA
                const int t = blockIdx.x + static_cast<int>(u / n_chunks) * gridDim.x, c = static_cast<int>(u % n_chunks);
                if (t >= p.n_tiles) return;
                const uint32_t sb = u % p.stg_bufs;
                int rows_in;
                const int boxes = boxes_of(t, c, &rows_in);
                if (lane == 0) mbar_expect_tx(&stg_free_bar[sb], static_cast<uint32_t>(boxes) * p.tw * p.out_box_rows * 128u);
                __syncwarp();
#pragma unroll 1
                for (int it = lane; it < boxes; it += 32) {
                    uint8_t* sm;
                    int c0, c1, c2, c3;
                    box_args(t, c, it, rows_in, sb, &sm, &c0, &c1, &c2, &c3);
                    tma_load_4d(sm, &p.tmr, &stg_free_bar[sb], c0, c1, c2, c3);
                }
            };
            if (has_res)
#pragma unroll 1
                for (int u = 0; u < p.stg_bufs; u++) fetch_residual(u);
            uint32_t u = 0;
            bool ok = true;
#pragma unroll 1
            for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x) {
#pragma unroll 1
                for (int c = 0; c < n_chunks && ok; c++, u++) {
                    const uint32_t sb = u % p.stg_bufs, ph = (u / p.stg_bufs) & 1u;
                    ok = mbar_wait_warp(&stg_full_bar[sb], ph, abort_flag, p.status, 0xa00 | (blockIdx.x << 12));
                    if (!ok) break;
                    int rows_in;
                    const int boxes = boxes_of(t, c, &rows_in);
                    bool mine = false;
#pragma unroll 1
                    for (int it = lane; it < boxes; it += 32) {
                        uint8_t* sm;
                        int c0, c1, c2, c3;
                        box_args(t, c, it, rows_in, sb, &sm, &c0, &c1, &c2, &c3);
                        tma_store_4d(&p.tmy, sm, c0, c1, c2, c3);
                        mine = true;
                    }
                    if (mine) {
                        tma_store_commit();
                        tma_store_wait_read();  // the boxes have been read: the buffer may take the next residual / chunk
                    }
                    __syncwarp();
                    if (has_res) fetch_residual(u + p.stg_bufs);
                    else if (lane == 0) mbar_arrive(&stg_free_bar[sb]);
                }
            }
            tma_store_wait_all();
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) {
        if (abort_s) __nanosleep(20000);  // let copies in flight land before the CTA retires
        tc_fence_after_sync();
        tmem_dealloc(tmem_base_s, 512);
    }
}

typedef void (*ChainKernel)(const ChainParams);
ChainKernel kernel_of(int out_mode) {
    return out_mode == OUT_STAGE ? chain_tc_kernel<OUT_STAGE> : (out_mode == OUT_POOL ? chain_tc_kernel<OUT_POOL> : chain_tc_kernel<OUT_DIRECT>);
}

int planes_of(int c) { return (c + 63) / 64; }
int pad16(int c) { return (c + 15) / 16 * 16; }
int round_up(int v, int a) { return (v + a - 1) / a * a; }

struct WeightBox {
    int tg, kg, rank4, bytes;
};

// Taps and K chunks per weight TMA box: as many as fit the target size, whole kernel rows first.
WeightBox weight_box(int cin, int k, int chunk, bool exact) {
    WeightBox w;
    const int kchunks = planes_of(cin);
    w.rank4 = (cin % 64 == 0) ? 1 : 0;
    w.tg = 1;
    for (int t : {k * k, k}) {
        if (t * chunk * 128 <= kWeightOpBytes) { w.tg = t; break; }
    }
    w.kg = 1;
    if (w.rank4 && (w.tg == k * k || k == 1)) w.kg = std::max(1, std::min(kchunks, kWeightOpBytes / (w.tg * chunk * 128)));
    // resident slabs are laid out back to back: a box must not reach past the layer's last K chunk
    while (exact && kchunks % w.kg) w.kg--;
    w.bytes = w.tg * w.kg * chunk * 128;
    return w;
}

struct LayerGeom {
    int qs, range, nb, n_pad, n_chunks, chunk_n, slot, per_pass, bgroups, col0, half_cols, in_dense, out_dense;
    int reach;   // rows past a block's own that its farthest tap reads
    int w_off;   // resident weights: offset of the layer's slabs
    WeightBox wb;
};

// Everything that follows from (chain, tile size, input slots, output mode, ring depth): per-layer geometry and the
// shared-memory layout.  Used by the tiler (to test what fits and to estimate the cost) and by the launcher.
struct Layout {
    LayerGeom g[kMaxChain];
    int halo, pitch, rows, out_dense;
    int in_planes, in_slot_bytes, in_off;
    int act_off[2], act_plane_bytes[2];
    int stg_off, stg_bufs, stg_planes, stg_plane_bytes, stg_buf_bytes, stg_base8;
    int ring_off, stage_bytes, bias_off, bias_floats, w_resident_bytes;
    size_t bytes;
    bool ok;
};

Layout make_layout(const ChainArgs& a, int th, int tw, int in_slots, int out_mode, int stg_bufs, int stages) {
    Layout y;
    std::memset(&y, 0, sizeof(y));
    const int L = a.n_layers;
    int halo = 0, last3 = -1;
    for (int l = 0; l < L; l++) {
        halo += a.k[l] / 2;
        if (a.k[l] == 3) last3 = l;
    }
    y.halo = halo;
    y.rows = th + 2 * halo;
    y.pitch = tw + 2 * halo;
    y.out_dense = last3 < L - 1 ? 1 : 0;   // 1x1 layers behind the last 3x3 one (or no 3x3 layer at all: frame = tile)
    int cum = 0, stage_bytes = 0, boff = 0, w_total = 0;
    for (int l = 0; l < L; l++) {
        LayerGeom& g = y.g[l];
        const int pad = a.k[l] / 2;
        cum += pad;
        g.in_dense = (l > last3 && halo > 0) ? 1 : 0;
        g.out_dense = (l >= last3 && l < L - 1 && halo > 0) ? 1 : 0;
        if (g.in_dense) {
            g.qs = 0;
            g.range = th * tw;
            g.reach = 0;
        } else {
            g.qs = cum * y.pitch + cum;
            g.range = (y.rows - 2 * cum - 1) * y.pitch + (y.pitch - 2 * cum);
            g.reach = pad * y.pitch + pad;
        }
        g.nb = (g.range + 127) / 128;
        g.n_pad = pad16(a.cout[l]);
        const bool last = l == L - 1;
        g.half_cols = (L == 1) ? 256 : 128;
        g.col0 = (last && L > 1) ? 256 : 0;
        g.n_chunks = (g.n_pad + g.half_cols - 1) / g.half_cols;
        g.chunk_n = g.n_chunks == 1 ? g.n_pad : g.half_cols;
        g.slot = round_up(std::min(g.chunk_n, g.n_pad), 32);
        g.per_pass = g.half_cols / g.slot;
        g.bgroups = (g.nb + g.per_pass - 1) / g.per_pass;
        g.wb = weight_box(a.cin[l], a.k[l], g.chunk_n, stages == 0);
        stage_bytes = std::max(stage_bytes, g.wb.bytes);
        g.w_off = w_total;
        w_total += g.n_chunks * planes_of(a.cin[l]) * a.k[l] * a.k[l] * g.chunk_n * 128;
        boff += g.n_pad;
    }
    y.bias_floats = boff;
    y.stage_bytes = stage_bytes;
    // shared memory: input slots, the two operand buffers, the staging tile(s), the weight ring, the biases.  The tensor core
    // always reads 128 rows per block (plus a tap's reach): past a buffer's last written row it reads on into whatever
    // follows (those accumulator rows are never used), which must still be this CTA's shared memory.
    size_t off = 0, read_end = 0;
    y.in_planes = planes_of(a.cin[0]);
    y.in_slot_bytes = round_up(y.rows * y.pitch, 8) * 128;
    y.in_off = 0;
    off = static_cast<size_t>(in_slots) * y.in_slot_bytes;
    read_end = std::max(read_end, off - y.in_slot_bytes + static_cast<size_t>(y.g[0].qs + y.g[0].nb * 128 + y.g[0].reach) * 128);
    for (int b = 0; b < 2; b++) {
        int planes = 0, rows_w = 0, rows_r = 0;
        for (int l = b; l < L - 1; l += 2) {
            const LayerGeom& g = y.g[l];
            planes = std::max(planes, planes_of(g.n_pad));
            rows_w = std::max(rows_w, g.out_dense ? th * tw : g.qs + g.range);
            const LayerGeom& r = y.g[l + 1];
            rows_r = std::max(rows_r, r.qs + r.nb * 128 + r.reach);
        }
        y.act_off[b] = static_cast<int>(off);
        y.act_plane_bytes[b] = round_up(rows_w, 8) * 128;
        off += static_cast<size_t>(planes) * y.act_plane_bytes[b];
        if (planes) read_end = std::max(read_end, off - y.act_plane_bytes[b] + static_cast<size_t>(rows_r) * 128);
    }
    const LayerGeom& z = y.g[L - 1];
    y.stg_off = static_cast<int>(off);
    y.stg_base8 = z.qs & ~7;
    if (out_mode == OUT_STAGE) {
        if (z.bgroups != 1) return y;   // a chunk's blocks must be one pass: the staged tile leaves as a whole
        y.stg_bufs = stg_bufs;
        y.stg_planes = planes_of(std::min(z.chunk_n, z.n_pad));
    } else if (out_mode == OUT_POOL) {
        y.stg_bufs = 1;
        y.stg_planes = planes_of(z.n_pad);
    }
    y.stg_plane_bytes = round_up(z.qs - y.stg_base8 + z.range, 8) * 128;
    y.stg_buf_bytes = y.stg_planes * y.stg_plane_bytes;
    off += static_cast<size_t>(y.stg_bufs) * y.stg_buf_bytes;
    y.ring_off = static_cast<int>(off);
    y.w_resident_bytes = w_total;
    off += stages == 0 ? static_cast<size_t>(w_total) : static_cast<size_t>(stages) * stage_bytes;
    y.bias_off = static_cast<int>(off);
    off += static_cast<size_t>(boff) * 4;
    y.bytes = std::max(off, read_end) + 1024;   // + what aligning the dynamic segment to 1024 bytes may cost
    y.ok = y.bytes <= static_cast<size_t>(kMaxSmem) && boff <= kMaxBias;
    return y;
}

std::vector<int> tile_candidates(int extent, bool even) {
    std::vector<int> v;
    for (int parts = 1; parts <= 16; parts++) {
        int t = (extent + parts - 1) / parts;
        if (even) t = (t + 1) / 2 * 2;
        if (t >= 1) v.push_back(t);
    }
    for (int t : {2, 4, 8, 16, 32, 64}) v.push_back(t);
    std::sort(v.begin(), v.end());
    v.erase(std::unique(v.begin(), v.end()), v.end());
    return v;
}

}  // namespace

bool chain_tc_layer_supported(int cin, int cout, int k) {
    return (k == 1 || k == 3) && cin % 8 == 0 && cout % 8 == 0 && cin >= 8 && cout >= 8 && cout <= 2048 && cin <= 2048;
}

// Picks the output tile from the SM count (Sec. IV-B: more cores -> smaller tiles -> more
// recomputed halo).  Among the tile shapes and buffer arrangements that fit in shared memory, takes the
// least estimated time = waves x per-tile time, the per-tile time being modelled in SM clocks from the
// UMMA issue rate (operand reads from shared memory vs. math), the epilogues, the hand-over between
// layers and the copies into shared memory.
ChainTiling chain_tc_tiling(const ChainArgs& a, int sm_count, int device_sms) {
    ChainTiling best{};
    best.ok = false;
    (void)device_sms;
    if (a.n_layers < 1 || a.n_layers > kMaxChain || sm_count < 1) return best;
    int halo = 0;
    for (int l = 0; l < a.n_layers; l++) {
        if (!chain_tc_layer_supported(a.cin[l], a.cout[l], a.k[l])) return best;
        if (l > 0 && a.cin[l] != a.cout[l - 1]) return best;
        halo += a.k[l] / 2;
    }
    const int L = a.n_layers;
    const int in_planes = planes_of(a.cin[0]);
    const std::vector<int> cand_h = tile_candidates(a.H, a.pool != 0);
    std::vector<int> cand_w = tile_candidates(a.W, a.pool != 0);
    // tile widths whose frame pitch is a multiple of 8 rows: a shifted operand window whose first row is not a
    // multiple of 8 rows into the tile straddles two swizzle atoms per 8-row group and costs the tensor core about
    // twice the shared-memory reads (measured: 85-90 cycles per N = 64 UMMA instead of 48); with such a pitch the
    // taps of the centre column start on atom boundaries
    for (int pitch8 = 8; pitch8 <= 256; pitch8 += 8) {
        const int tw8 = pitch8 - 2 * halo;
        if (tw8 >= 2 && tw8 <= a.W && (!a.pool || tw8 % 2 == 0)) cand_w.push_back(tw8);
    }
    std::sort(cand_w.begin(), cand_w.end());
    cand_w.erase(std::unique(cand_w.begin(), cand_w.end()), cand_w.end());
    // input arrangements: the whole frame resident (two frames: the next tile's is prefetched), or - for a 1x1 first
    // layer - a ring of planes released one by one, in rounds of `group` planes (a divisor of the plane count)
    struct InMode { int ring, group, slots; };
    std::vector<InMode> in_modes;
    if (a.k[0] == 1) {
        for (int g = std::min(in_planes, 8); g >= 1; g--)
            if (in_planes % g == 0 && 2 * g <= kMaxInSlots) in_modes.push_back({1, g, 2 * g});
    }
    if (in_planes <= kMaxInSlots) {
        if (2 * in_planes <= kMaxInSlots) in_modes.push_back({0, in_planes, 2 * in_planes});
        in_modes.push_back({0, in_planes, in_planes});
    }
    struct OutChoice { int mode, bufs; };
    std::vector<OutChoice> out_modes;
    if (a.pool) out_modes.push_back({OUT_POOL, 1});
    else { out_modes.push_back({OUT_STAGE, 2}); out_modes.push_back({OUT_STAGE, 1}); out_modes.push_back({OUT_DIRECT, 0}); }
    for (int th : cand_h)
        for (int tw : cand_w) {
            const int rows = th + 2 * halo, pitch = tw + 2 * halo;
            if (rows > 256 || pitch > 256 || th > 256 || tw > 256) continue;
#ifdef DLF_TRACE
            if (const char* force = getenv("DLF_CHAIN_TILE")) {   // trace builds only: "th,tw[,out_mode]"
                int fth = 0, ftw = 0;
                if (sscanf(force, "%d,%d", &fth, &ftw) == 2 && (fth != th || ftw != tw)) continue;
            }
#endif
            const int tiles_h = (a.H + th - 1) / th, tiles_w = (a.W + tw - 1) / tw;
            const long long n_tiles = static_cast<long long>(a.N) * tiles_h * tiles_w;
            if (n_tiles > 0x7fffffffLL) continue;
            const long long waves = (n_tiles + sm_count - 1) / sm_count;
            for (const OutChoice& oc : out_modes)
                for (const InMode& im : in_modes) {
                    // the deepest weight ring that fits (an even stage count; four producers take a multiple of four)
                    Layout y;
                    int stages = 0;
                    for (int st : {0, 8, 6, 4, 2}) {   // 0: all weights resident
                        y = make_layout(a, th, tw, im.slots, oc.mode, oc.bufs, st);
                        if (y.ok) { stages = st; break; }
                        if (y.stg_bufs == 0 && oc.mode == OUT_STAGE) break;   // not stageable at this tile size
                    }
                    if (!y.ok) continue;
                    // Per-tile time in SM clocks, from what was measured on B200.  Every role of this kernel is bound by
                    // its own instruction stream (about 4 cycles per instruction of a lone warp): the issuing warp spends
                    // about 150 cycles per weight slab group it walks (1500 when the slab comes through the ring: measured on
                    // ResNet bottleneck spans, where a ring of four to six boxes runs dry and every box then costs most of a
                    // TMA round trip - the same spans run 1.3 to 1.7 times faster with resident weights) plus 25 per UMMA, unless the tensor core needs longer (operand reads from shared memory vs.
                    // math); a layer can start about 900 cycles after its predecessor's last instruction at the earliest
                    // (commit, fences, wake-ups) plus the drain of the last pass; a pair of epilogue warps turns a 128 x 64
                    // piece of an accumulator into fp16 in 1200 (operand tile) to 3300 (staged output with a residual)
                    // cycles; the weight ring delivers its own size per TMA round trip.
                    double chain = 0.0, epi_last_clk = 0.0, w_bytes = 0.0, useful = 0.0, computed = 0.0, in_reloads = 1.0;
                    for (int l = 0; l < L; l++) {
                        const LayerGeom& g = y.g[l];
                        const int ksteps = a.k[l] * a.k[l] * ((a.cin[l] + 15) / 16);
                        const int passes = g.n_chunks * g.bgroups;
                        const int boxes = passes * (a.k[l] * a.k[l] / g.wb.tg) * ((planes_of(a.cin[l]) + g.wb.kg - 1) / g.wb.kg);
                        double tensor = 0.0;
                        for (int ch = 0; ch < g.n_chunks; ch++) {
                            const int n = std::min(g.chunk_n, g.n_pad - ch * g.chunk_n);
                            // operand reads from shared memory: 4 KB of pixels (8 KB where the window straddles swizzle
                            // atoms: every tap of a 3x3 layer but the centre column's at a pitch that is a multiple of 8,
                            // else all but the centre tap) and n x 32 bytes of weights, at 128 bytes per clock
                            const double straddle = (a.k[l] == 1 || g.in_dense) ? 0.0 : (pitch % 8 == 0 ? 6.0 / 9.0 : 8.0 / 9.0);
                            tensor += static_cast<double>(g.nb) * ksteps * (std::max(32.0 * (1.0 + straddle) + n / 4.0, n / 2.0) + 6.0);
                        }
                        const double issue = boxes * (stages == 0 ? 150.0 : 1500.0) + 25.0 * g.n_chunks * g.nb * ksteps;
                        const double mma = std::max(issue, tensor);
                        const double units = static_cast<double>(g.nb) * ((g.n_pad + 63) / 64);   // 128 x 32 pieces per warp of a group
                        if (l < L - 1) {
                            // the next layer starts when this one's last pass has been drained and handed over
                            const double epi = units * 1200.0;
                            chain += std::max(mma, epi * (passes - 1) / passes) + epi / passes + 900.0;
                        } else {
                            chain += mma;
                            epi_last_clk = units * (oc.mode == OUT_DIRECT ? 6500.0 : (a.res ? 3300.0 : 2600.0)) + (oc.mode == OUT_POOL ? units * 1200.0 : 0.0) + 400.0;
                        }
                        w_bytes += static_cast<double>(g.bgroups) * a.k[l] * a.k[l] * round_up(a.cin[l], 64) * g.n_pad * 2.0;
                        if (l == 0 && im.ring) in_reloads = passes;
                        computed += static_cast<double>(g.nb) * 128.0 * a.k[l] * a.k[l] * a.cin[l] * a.cout[l];
                        useful += static_cast<double>(std::min(th, a.H)) * std::min(tw, a.W) * a.k[l] * a.k[l] * a.cin[l] * a.cout[l];
                    }
                    const double load_in = static_cast<double>(rows) * pitch * in_planes * 128.0 * in_reloads / 48.0;
                    const double load_w = stages == 0 ? 0.0 : w_bytes * 2200.0 / (static_cast<double>(stages) * y.stage_bytes);
                    double clk = std::max(std::max(chain, epi_last_clk), load_w) + 300.0;
                    // a single input frame is loaded between two tiles; a second frame / a plane ring hides the load
                    clk = (im.slots > in_planes || im.ring) ? std::max(clk, load_in) : clk + load_in + 1500.0;
                    if (oc.mode == OUT_STAGE && oc.bufs == 1) clk += 600.0;
                    // (among tilings of equal time the one that recomputes less wins: it loads less and leaves SMs free)
                    const double cost = (static_cast<double>(waves) * clk + epi_last_clk + 3000.0 + (stages == 0 ? y.w_resident_bytes / 48.0 : 0.0)) *
                                        (1.0 + 0.01 * (computed / useful - 1.0));
#ifdef DLF_TRACE
                    if (getenv("DLF_TILER_LIST"))
                        fprintf(stderr, "tile %dx%d in(%d,%d,%d) out(%d,%d) stages %d waves %lld chain %.0f epi_last %.0f load_w %.0f load_in %.0f clk %.0f red %.2f cost %.0f\n", th, tw,
                                im.ring, im.group, im.slots, oc.mode, oc.bufs, stages, waves, chain, epi_last_clk, load_w, load_in, clk, computed / useful, cost);
#endif
                    if (!best.ok || cost < best.cost) {
                        best.th = th; best.tw = tw; best.halo = halo; best.pitch = pitch; best.rows = rows;
                        best.tiles_h = tiles_h; best.tiles_w = tiles_w; best.n_tiles = static_cast<int>(n_tiles);
                        best.in_ring = im.ring; best.in_group = im.group; best.in_slots = im.slots;
                        best.out_mode = oc.mode; best.stg_bufs = y.stg_bufs;
                        best.stages = stages; best.stage_bytes = y.stage_bytes;
                        best.smem_bytes = y.bytes;
                        best.redundancy = computed / useful;
                        best.cost = cost;
                        best.ok = true;
                    }
                }
        }
    return best;
}

int launch_chain_tc(const ChainArgs& a, const ChainTiling& t, int sm_count, int* status_dev, cudaStream_t s) {
    if (!t.ok) return DLF_E_PLAN;
    {
        int rc = chain_tc_init();
        if (rc) return rc;
    }
    const Layout y = make_layout(a, t.th, t.tw, t.in_slots, t.out_mode, t.stg_bufs, t.stages);
    if (!y.ok) return DLF_E_PLAN;
    ChainParams p;
    std::memset(&p, 0, sizeof(p));
    const int nl = a.n_layers;
    p.n_layers = nl;
    p.N = a.N; p.H = a.H; p.W = a.W;
    p.th = t.th; p.tw = t.tw; p.halo = y.halo; p.pitch = y.pitch; p.rows = y.rows;
    p.tiles_h = t.tiles_h; p.tiles_w = t.tiles_w; p.n_tiles = t.n_tiles;
    p.in_planes = y.in_planes; p.in_group = t.in_group; p.in_slots = t.in_slots; p.in_ring = t.in_ring;
    p.in_slot_bytes = y.in_slot_bytes; p.in_off = y.in_off;
    for (int b = 0; b < 2; b++) { p.act_off[b] = y.act_off[b]; p.act_plane_bytes[b] = y.act_plane_bytes[b]; }
    p.out_mode = t.out_mode; p.out_dense = y.out_dense; p.out_box_rows = y.out_dense ? t.th : 1;
    p.stg_off = y.stg_off; p.stg_bufs = std::max(1, y.stg_bufs); p.stg_buf_bytes = y.stg_buf_bytes; p.stg_plane_bytes = y.stg_plane_bytes;
    p.stg_base8 = y.stg_base8;
    p.ring_off = y.ring_off; p.stages = t.stages; p.stage_bytes = y.stage_bytes;
    p.w_producers = (t.stages % 4 == 0) ? kWeightWarps : 2;
    p.bias_off = y.bias_off; p.bias_floats = y.bias_floats;
    int boff = 0;
    for (int l = 0; l < nl; l++) {
        ChainLayerP& L = p.L[l];
        const LayerGeom& g = y.g[l];
        L.cin = a.cin[l]; L.cout = a.cout[l]; L.k = a.k[l]; L.pad = a.k[l] / 2; L.act = a.act[l];
        L.kchunks = planes_of(a.cin[l]);
        L.ksteps_last = ((a.cin[l] - (L.kchunks - 1) * 64) + 15) / 16;
        L.qs = g.qs; L.range = g.range; L.nb = g.nb; L.n_pad = g.n_pad; L.n_chunks = g.n_chunks; L.chunk_n = g.chunk_n;
        L.slot = g.slot; L.per_pass = g.per_pass; L.bgroups = g.bgroups;
        L.col0 = g.col0; L.half_cols = g.half_cols; L.in_dense = g.in_dense; L.out_dense = g.out_dense;
        L.bias_off = boff;
        boff += g.n_pad;
        L.bias = a.bias[l];
        L.tg = g.wb.tg; L.kg = g.wb.kg; L.w_rank4 = g.wb.rank4; L.w_off = g.w_off;
        const uint64_t taps = static_cast<uint64_t>(a.k[l]) * a.k[l];
        const uint32_t box_n = static_cast<uint32_t>(std::min(g.chunk_n, g.n_pad));
        int rc;
        if (g.wb.rank4) {  // [cout][tap][cin] seen as (64 channels, cout, tap, cin / 64)
            const uint64_t dims[4] = {64, static_cast<uint64_t>(a.cout[l]), taps, static_cast<uint64_t>(a.cin[l] / 64)};
            const uint64_t strides[3] = {taps * a.cin[l] * 2, static_cast<uint64_t>(a.cin[l]) * 2, 128};
            const uint32_t box[4] = {64, box_n, static_cast<uint32_t>(g.wb.tg), static_cast<uint32_t>(g.wb.kg)};
            const uint32_t es[4] = {1, 1, 1, 1};
            rc = encode_tmap(&p.tmw[l], a.w[l], 4, dims, strides, box, es);
        } else {         // (cin, cout, tap): K chunks are addressed along dimension 0, zero-filled past cin
            const uint64_t dims[3] = {static_cast<uint64_t>(a.cin[l]), static_cast<uint64_t>(a.cout[l]), taps};
            const uint64_t strides[2] = {taps * a.cin[l] * 2, static_cast<uint64_t>(a.cin[l]) * 2};
            const uint32_t box[3] = {64, box_n, static_cast<uint32_t>(g.wb.tg)};
            const uint32_t es[3] = {1, 1, 1};
            rc = encode_tmap(&p.tmw[l], a.w[l], 3, dims, strides, box, es);
        }
        if (rc) return rc;
    }
    p.pool = a.pool;
    p.cout_last = a.cout[nl - 1];
    p.res = static_cast<const __half*>(a.res);
    p.out = static_cast<__half*>(a.y);
    p.status = status_dev;
    {
        const uint64_t dims[4] = {static_cast<uint64_t>(a.cin[0]), static_cast<uint64_t>(a.W), static_cast<uint64_t>(a.H),
                                  static_cast<uint64_t>(a.N)};
        const uint64_t strides[3] = {static_cast<uint64_t>(a.cin[0]) * 2, static_cast<uint64_t>(a.W) * a.cin[0] * 2,
                                     static_cast<uint64_t>(a.H) * a.W * a.cin[0] * 2};
        const uint32_t box[4] = {64, static_cast<uint32_t>(y.pitch), static_cast<uint32_t>(y.rows), 1};
        const uint32_t es[4] = {1, 1, 1, 1};
        int rc = encode_tmap(&p.tmx, a.x, 4, dims, strides, box, es);
        if (rc) return rc;
    }
    if (t.out_mode == OUT_STAGE) {   // output / residual tile: a 64-channel plane of the dense tile, or of one of its rows
        const int co = p.cout_last;
        const uint64_t dims[4] = {static_cast<uint64_t>(co), static_cast<uint64_t>(a.W), static_cast<uint64_t>(a.H), static_cast<uint64_t>(a.N)};
        const uint64_t strides[3] = {static_cast<uint64_t>(co) * 2, static_cast<uint64_t>(a.W) * co * 2, static_cast<uint64_t>(a.H) * a.W * co * 2};
        const uint32_t box[4] = {64, static_cast<uint32_t>(t.tw), static_cast<uint32_t>(p.out_box_rows), 1};
        const uint32_t es[4] = {1, 1, 1, 1};
        int rc = encode_tmap(&p.tmy, a.y, 4, dims, strides, box, es);
        if (rc) return rc;
        p.tmr = p.tmy;
        if (a.res) {
            rc = encode_tmap(&p.tmr, a.res, 4, dims, strides, box, es);
            if (rc) return rc;
        }
    }
    const int grid = std::max(1, std::min(sm_count, t.n_tiles));
    const size_t smem = std::max<size_t>(y.bytes, 120 * 1024);   // never two of these CTAs on an SM: each holds all of tensor memory
#ifdef DLF_TRACE
    fprintf(stderr, "chain_tc: L=%d tile %dx%d frame %dx%d tiles %d grid %d in ring %d group %d slots %d out mode %d bufs %d stages %d stage_bytes %d smem %zu red %.2f\n",
            nl, t.th, t.tw, y.rows, y.pitch, t.n_tiles, grid, t.in_ring, t.in_group, t.in_slots, t.out_mode, y.stg_bufs, t.stages, y.stage_bytes, y.bytes, t.redundancy);
    for (int l = 0; l < nl; l++)
        fprintf(stderr, "  layer %d: %d->%d k%d nb %d chunks %d x %d per_pass %d tg %d kg %d dense in %d out %d\n", l, a.cin[l], a.cout[l], a.k[l], p.L[l].nb,
                p.L[l].n_chunks, p.L[l].chunk_n, p.L[l].per_pass, p.L[l].tg, p.L[l].kg, p.L[l].in_dense, p.L[l].out_dense);
#endif
    cudaError_t e = launch_kernel(kernel_of(t.out_mode), grid, kThreads, smem, s, p);
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

int chain_tc_init() {
    static bool attr_set[kMaxDevices] = {};
    const int dev = current_device_slot();
    if (dev < 0) return DLF_E_UNSUPPORTED;
    if (!attr_set[dev]) {
        for (int mode = OUT_DIRECT; mode <= OUT_POOL; mode++) {
            cudaError_t e = cudaFuncSetAttribute(kernel_of(mode), cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
            if (e != cudaSuccess) return cuda_fail(e);
        }
        attr_set[dev] = true;
    }
    return DLF_OK;
}

}  // namespace dlf
