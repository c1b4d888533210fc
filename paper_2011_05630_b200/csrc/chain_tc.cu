// Fused fusion-group kernel: a chain of stride-1, size-keeping dense convolutions (3x3 pad 1 or
// 1x1) with bias / activation after each, optional residual and 2x2 max-pool on the last one,
// executed by ONE kernel whose intermediate feature maps never leave the SM (Sec. III-B of the
// paper: a fused layer's output is produced on chip and reused at once; Sec. IV-B: a spatial
// tile of a fused block recomputes its halo).  With one layer it is also the library's general
// stride-1 convolution kernel: the input tile is read once instead of once per tap.
//
// Work item = (image, output tile th x tw of the last layer).  The tile's receptive-field frame
// (th + 2 halo) x (tw + 2 halo), halo = sum of the paddings, is loaded ONCE by TMA (zero fill
// outside the image = the first layer's padding) as a pixel-linear buffer: row q = fy*pitch + fx
// holds one pixel's 64 channels (128 bytes, 128-byte swizzle); wider layers use several planes.
// In that layout tap (r, s) of a 3x3 layer is the same buffer shifted by (r-1)*pitch + (s-1)
// rows, so every layer - the first included - feeds the tensor cores straight from the resident
// tile through a shifted shared-memory descriptor: no im2col, no per-tap reload.  A layer's M
// dimension is the linear range of frame positions it must produce (wrap-around columns are
// computed and ignored), cut into 128-row blocks; output channels are cut into chunks of at
// most 256.  A pass = (layer, channel chunk, group of blocks) accumulates in one half of tensor
// memory while the four epilogue warps drain the other half: bias, residual, activation, fp16
// rounding, then either the next layer's operand tile in shared memory (positions outside the
// image forced to zero: they are the next layer's padding) or, for the group's last layer,
// global memory.  Weights stream through a TMA ring, once per pass; the next tile's input frame
// is prefetched into a second buffer while the current tile computes.
//
// Warp roles: 0-7 epilogue (two per TMEM lane quarter, alternating 32-column chunks), 8 UMMA
// issuer, 9-10 weight producers, 11 input producer.  Measured on B200: one TMA instruction
// keeps its issuing thread busy for about 0.28 us whatever the box size, so weights travel in
// boxes of several taps / K chunks (up to 32 KB) and the loads are spread over several warps.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <vector>

#include "internal.h"
#include "ptx.cuh"

namespace dlf {

namespace {

constexpr int kEpiWarps = 8;                 // warps 0..7: epilogue (warp & 3 = TMEM lane quarter)
constexpr int kMmaWarp = kEpiWarps;          // warp 8: UMMA issuer, owns the TMEM allocation
constexpr int kWeightWarp0 = kEpiWarps + 1;  // warps 9, 10: weight producers (alternate ring stages)
constexpr int kInputWarp0 = kEpiWarps + 3;   // warp 11: input producer (one box per 64-channel plane, a tile ahead)
constexpr int kThreads = 32 * (kEpiWarps + 4);
constexpr int kWeightOpBytes = 32 * 1024;    // target size of one weight TMA box
constexpr int kMaxSmem = 232448 - 1024;  // dynamic part: the 227 KB per-CTA limit minus the static barriers
constexpr int kMaxBias = 4096;           // floats of bias staged in shared memory (all layers)

struct ChainLayerP {
    int cin, cout, k, pad, act;
    int kchunks, ksteps_last;  // 64-channel K chunks; 16-channel steps in the last one
    int qs, range, nb;         // first frame row produced, rows produced, 128-row blocks
    int n_pad;                 // cout rounded up to 16
    int n_chunks, chunk_n;     // channel chunks of chunk_n (the last one may be smaller)
    int slot, per_pass;        // TMEM columns per block, blocks per pass (half of TMEM)
    int tg, kg, w_rank4;       // taps and K chunks per weight box; 4-d weight view (cin % 64 == 0)
    int bias_off;
    const float* bias;
};

struct ChainParams {
    CUtensorMap tmx;
    CUtensorMap tmw[kMaxChain];
    ChainLayerP L[kMaxChain];
    int n_layers;
    int N, H, W;
    int th, tw, halo, pitch, rows;  // frame geometry
    int tiles_h, tiles_w, n_tiles;
    int plane_bytes;                // rows_alloc * 128
    int in_planes, in_bufs, in_buf_bytes;
    int act_off, act_buf_bytes;
    int ring_off, stages, stage_bytes;
    int bias_off, bias_floats;
    int pool;
    int cout_last;
    const __half* res;
    __half* out;
    int* status;
};

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory"); }

__device__ __forceinline__ int chunk_cols(const ChainLayerP& L, int c) {
    return min(L.chunk_n, L.n_pad - c * L.chunk_n);
}

struct EpiCtx {
    int row, half;            // TMEM lane of this thread; which alternating 32-column chunks it takes
    uint32_t tmem_lane, tmem_col;
    int gy0, gx0, n;          // image coordinates of frame row 0 / column 0, image index
    int b0, nblk, ncols, ch0; // blocks of this pass, columns and first channel of this chunk
    uint8_t* obuf;
    const float* bl;
    __half2 act_lo, act_hi;   // applied to rounded pairs
};

// Drains one pass.  MODE 0: next layer's operand tile in shared memory (zero outside the image);
// 1: global memory; 2: global memory with residual; 3: shared staging tile with residual (pooled
// last layer).  The activation is a clamp to [act_lo, act_hi] (none: -inf..inf, ReLU: 0..inf,
// ReLU6: 0..6), which keeps the loop free of branches without one copy of the code per activation.
template <int MODE>
__device__ __forceinline__ void epi_pass(const ChainParams& p, const ChainLayerP& L, const EpiCtx& cx) {
    constexpr bool kGlobal = (MODE == 1 || MODE == 2);
    constexpr bool kRes = (MODE == 2 || MODE == 3);
    for (int b = 0; b < cx.nblk; b++) {
        const int q = L.qs + (cx.b0 + b) * 128 + cx.row;
        const int fy = q / p.pitch, fx = q - fy * p.pitch;
        const int gy = cx.gy0 + fy, gx = cx.gx0 + fx;
        const bool in_img = gy >= 0 && gy < p.H && gx >= 0 && gx < p.W;
        const bool in_tile = fy >= p.halo && fy < p.halo + p.th && fx >= p.halo && fx < p.halo + p.tw;
        const bool live = q < L.qs + L.range && (!kGlobal || (in_img && in_tile));
        const long long gpix = (static_cast<long long>(cx.n) * p.H + gy) * p.W + gx;
        const uint32_t taddr = cx.tmem_lane + cx.tmem_col + b * L.slot;
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
                uint4 val = make_uint4(0u, 0u, 0u, 0u);
                if (kGlobal || in_img) {
                    float a[8];
                    const float4 b0 = *reinterpret_cast<const float4*>(cx.bl + co);
                    const float4 b1 = *reinterpret_cast<const float4*>(cx.bl + co + 4);
                    a[0] = v[g * 8 + 0] + b0.x; a[1] = v[g * 8 + 1] + b0.y; a[2] = v[g * 8 + 2] + b0.z; a[3] = v[g * 8 + 3] + b0.w;
                    a[4] = v[g * 8 + 4] + b1.x; a[5] = v[g * 8 + 5] + b1.y; a[6] = v[g * 8 + 6] + b1.z; a[7] = v[g * 8 + 7] + b1.w;
                    if (kRes) {
                        if (co < L.cout && (kGlobal || in_tile)) {
                            const uint4 rv = __ldg(reinterpret_cast<const uint4*>(p.res + gpix * L.cout + co));
                            const __half2* rh = reinterpret_cast<const __half2*>(&rv);
#pragma unroll
                            for (int e = 0; e < 4; e++) {
                                const float2 rf = __half22float2(rh[e]);
                                a[2 * e] += rf.x;
                                a[2 * e + 1] += rf.y;
                            }
                        }
                    }
                    // channels past cout (padding up to 16) carry zero weights and zero bias: act(0) = 0,
                    // so the next layer's K padding stays zero
                    val.x = pack_half2_clamp(a[0], a[1], cx.act_lo, cx.act_hi);
                    val.y = pack_half2_clamp(a[2], a[3], cx.act_lo, cx.act_hi);
                    val.z = pack_half2_clamp(a[4], a[5], cx.act_lo, cx.act_hi);
                    val.w = pack_half2_clamp(a[6], a[7], cx.act_lo, cx.act_hi);
                }
                if (kGlobal) {
                    if (co < L.cout) *reinterpret_cast<uint4*>(p.out + gpix * L.cout + co) = val;
                } else {
                    const int g8 = co >> 3;  // 8-channel group index
                    *reinterpret_cast<uint4*>(cx.obuf + static_cast<size_t>(g8 >> 3) * p.plane_bytes + static_cast<size_t>(q) * 128 +
                                              (((g8 & 7) ^ (q & 7)) << 4)) = val;
                }
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1) chain_tc_kernel(const __grid_constant__ ChainParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t wfull_bar[8], wempty_bar[8], in_full_bar[2], in_empty_bar[2], acc_full_bar[2], acc_empty_bar[2],
        act_ready_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sbase = smem_raw + (base - smem_u32(smem_raw));
    float* bias_s = reinterpret_cast<float*>(sbase + p.bias_off);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = &abort_s;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int i = 0; i < p.stages; i++) {
            mbar_init(&wfull_bar[i], 1);
            mbar_init(&wempty_bar[i], 1);
        }
        for (int i = 0; i < 2; i++) {
            mbar_init(&in_full_bar[i], 1);
            mbar_init(&in_empty_bar[i], 1);
            mbar_init(&acc_full_bar[i], 1);
            mbar_init(&acc_empty_bar[i], kEpiWarps);
        }
        mbar_init(&act_ready_bar, kEpiWarps);
        fence_barrier_init();
        tma_prefetch_desc(&p.tmx);
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
    if (warp < kWeightWarp0 || warp >= kInputWarp0) pdl_wait();
    const uint32_t tmem_base = tmem_base_s;
    const int frame_rows = p.rows * p.pitch;

    if (warp >= kInputWarp0) {
        // ---- input producer: one frame per tile, prefetched into the free input buffer ---------
        if (lane == 0) {
            uint32_t tile_i = 0;
            for (int t = blockIdx.x; t < p.n_tiles; t += gridDim.x, tile_i++) {
                const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h, n = t / (p.tiles_w * p.tiles_h);
                const uint32_t ib = tile_i % p.in_bufs, ph = (tile_i / p.in_bufs) & 1u;
                if (!mbar_wait(&in_empty_bar[ib], ph ^ 1u, abort_flag, p.status, 0x100 | (blockIdx.x << 12))) break;
                mbar_expect_tx(&in_full_bar[ib], static_cast<uint32_t>(p.in_planes) * frame_rows * 128u);
                for (int pl = 0; pl < p.in_planes; pl++)
                    tma_load_4d(sbase + static_cast<size_t>(ib) * p.in_buf_bytes + static_cast<size_t>(pl) * p.plane_bytes, &p.tmx,
                                &in_full_bar[ib], pl * 64, txi * p.tw - p.halo, tyi * p.th - p.halo, n);
            }
        }
    } else if (warp >= kWeightWarp0) {
        // ---- weight producers: one box of tg taps x kg K chunks x [chunk_n][64] per ring stage ------
        if (lane == 0) {
            const uint32_t parity = warp - kWeightWarp0;
            uint32_t wit = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x) {
                for (int l = 0; l < p.n_layers && ok; l++) {
                    const ChainLayerP& L = p.L[l];
                    const int passes = (L.nb + L.per_pass - 1) / L.per_pass;
                    const uint32_t bytes = static_cast<uint32_t>(L.tg * L.kg * L.chunk_n) * 128u;  // the whole box
                    for (int c = 0; c < L.n_chunks && ok; c++)
                        for (int ps = 0; ps < passes && ok; ps++)
                            for (int t0 = 0; t0 < L.k * L.k && ok; t0 += L.tg)
                                for (int g0 = 0; g0 < L.kchunks; g0 += L.kg, wit++) {
                                    const int st = wit % p.stages;
                                    // a ring stage belongs to one producer (see the parity of mbarrier waits)
                                    if ((st & 1u) != parity) continue;
                                    ok = mbar_wait(&wempty_bar[st], ((wit / p.stages) & 1u) ^ 1u, abort_flag, p.status,
                                                   0x200 | (blockIdx.x << 12));
                                    if (!ok) break;
                                    mbar_expect_tx(&wfull_bar[st], bytes);
                                    uint8_t* dst = sbase + p.ring_off + static_cast<size_t>(st) * p.stage_bytes;
                                    if (L.w_rank4) tma_load_4d(dst, &p.tmw[l], &wfull_bar[st], 0, c * L.chunk_n, t0, g0);
                                    else tma_load_3d(dst, &p.tmw[l], &wfull_bar[st], g0 * 64, c * L.chunk_n, t0);
                                }
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ---- UMMA issuer: the whole warp walks the loops (warp-uniform addresses), one elected lane issues ----
        const uint64_t desc0 = umma_desc_sw128(0);
        uint32_t wit = 0, tile_i = 0, pass_i = 0, act_i = 0;
        bool ok = true;
        DLF_TRACE_DECL(tacc, tmark);  // cycles of CTA 0's issuer: 0 input wait, 1 layer hand-off wait, 2 accumulator wait, 3 weight wait, 4 issue
        for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x, tile_i++) {
            const uint32_t ib = tile_i % p.in_bufs;
            ok = mbar_wait_warp(&in_full_bar[ib], (tile_i / p.in_bufs) & 1u, abort_flag, p.status, 0x300 | (blockIdx.x << 12));
            if (!ok) break;
            DLF_TRACE_ACC(tacc, 0, tmark);
            for (int l = 0; l < p.n_layers && ok; l++) {
                const ChainLayerP& L = p.L[l];
                if (l > 0) {  // the epilogue has written all of the previous layer's tile
                    ok = mbar_wait_warp(&act_ready_bar, act_i & 1u, abort_flag, p.status, 0x400 | (blockIdx.x << 12));
                    if (!ok) break;
                    act_i++;
                    DLF_TRACE_ACC(tacc, 1, tmark);
                }
                const uint32_t abuf = l == 0 ? base + ib * p.in_buf_bytes : base + p.act_off + ((l - 1) & 1) * p.act_buf_bytes;
                const int taps = L.k * L.k;
                const uint32_t w_tap16 = static_cast<uint32_t>(L.chunk_n) * 8u;  // one tap's [chunk_n][64] slab, 16-byte units
                for (int c = 0; c < L.n_chunks && ok; c++) {
                    const uint32_t idesc = umma_idesc_f16(chunk_cols(L, c));
                    for (int b0 = 0; b0 < L.nb && ok; b0 += L.per_pass, pass_i++) {
                        const int nblk = min(L.per_pass, L.nb - b0);
                        const uint32_t half = pass_i & 1u;
                        ok = mbar_wait_warp(&acc_empty_bar[half], ((pass_i >> 1) & 1u) ^ 1u, abort_flag, p.status,
                                            0x500 | (blockIdx.x << 12));
                        if (!ok) break;
                        DLF_TRACE_ACC(tacc, 2, tmark);
                        tc_fence_after_sync();
                        const uint32_t d_tmem0 = tmem_base + half * 256u;
                        const uint32_t arow_base = abuf + (L.qs + b0 * 128) * 128;
                        for (int t0 = 0; t0 < taps && ok; t0 += L.tg) {
                            for (int g0 = 0; g0 < L.kchunks; g0 += L.kg, wit++) {
                                const int st = wit % p.stages;
                                ok = mbar_wait_warp(&wfull_bar[st], (wit / p.stages) & 1u, abort_flag, p.status,
                                                    0x600 | (blockIdx.x << 12));
                                if (!ok) break;
                                DLF_TRACE_ACC(tacc, 3, tmark);
                                tc_fence_after_sync();
                                const uint64_t wd0 = desc0 + ((base + p.ring_off + st * p.stage_bytes) >> 4);
                                const int g_end = min(L.kg, L.kchunks - g0);
                                if (elect_one()) {
                                    for (int g = 0; g < g_end; g++) {
                                        const int kc = g0 + g;
                                        const int ksteps = (kc == L.kchunks - 1) ? L.ksteps_last : 4;
                                        const uint32_t aplane = arow_base + kc * p.plane_bytes;
                                        for (int tt = 0; tt < L.tg; tt++) {
                                            const int tap = t0 + tt;
                                            const int r = tap / L.k, sx = tap - r * L.k;
                                            const int shift = (r - L.pad) * p.pitch + (sx - L.pad);
                                            const uint64_t bd = wd0 + static_cast<uint32_t>(g * L.tg + tt) * w_tap16;
                                            const uint32_t arow0 = aplane + shift * 128;
                                            uint64_t ad = desc0 + (arow0 >> 4);
                                            const uint32_t acc0 = (tap | kc) != 0;
                                            uint32_t d_tmem = d_tmem0;
                                            for (int b = 0; b < nblk; b++, d_tmem += L.slot, ad += (128 * 128) >> 4) {
                                                umma_f16(d_tmem, ad, bd, idesc, acc0);
                                                if (ksteps > 1) umma_f16(d_tmem, ad + 2, bd + 2, idesc, 1);
                                                if (ksteps > 2) umma_f16(d_tmem, ad + 4, bd + 4, idesc, 1);
                                                if (ksteps > 3) umma_f16(d_tmem, ad + 6, bd + 6, idesc, 1);
                                            }
                                        }
                                    }
                                    umma_commit(&wempty_bar[st]);
                                }
                                __syncwarp();
                                DLF_TRACE_ACC(tacc, 4, tmark);
                            }
                        }
                        if (ok && elect_one()) umma_commit(&acc_full_bar[half]);
                        __syncwarp();
                    }
                }
                // the input frame is read by the first layer only
                if (ok && l == 0 && elect_one()) umma_commit(&in_empty_bar[ib]);
                __syncwarp();
            }
        }
        if (lane == 0) DLF_TRACE_FLUSH_AT(p.status, tacc, 0);
    } else {
        // ---- epilogue warps ------------------------------------------------------------------------------------
        const int et = threadIdx.x;  // 0 .. 32*kEpiWarps-1
        // biases staged by the epilogue warps alone, behind the CTA-wide barrier: the producers' first copies do not
        // wait for these loads
        for (int l = 0; l < p.n_layers; l++) {
            const ChainLayerP& L = p.L[l];
            for (int i = et; i < L.n_pad; i += 32 * kEpiWarps) bias_s[L.bias_off + i] = i < L.cout ? __ldg(L.bias + i) : 0.0f;
        }
        epi_bar_sync();
        EpiCtx cx;
        cx.row = (warp & 3) * 32 + lane;
        cx.half = warp >> 2;
        cx.tmem_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        uint32_t pass_i = 0;
        bool ok = true;
        DLF_TRACE_DECL(eacc, emark);  // cycles of CTA 0's first epilogue thread: 0 accumulator wait, 1 + mode: drain, 5 pooled copy-out
        for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x) {
            const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h, n = t / (p.tiles_w * p.tiles_h);
            cx.gy0 = tyi * p.th - p.halo;
            cx.gx0 = txi * p.tw - p.halo;
            cx.n = n;
            for (int l = 0; l < p.n_layers && ok; l++) {
                const ChainLayerP& L = p.L[l];
                const bool last = (l == p.n_layers - 1);
                const int mode = (last && !p.pool) ? (p.res != nullptr ? 2 : 1) : ((last && p.res != nullptr) ? 3 : 0);
                cx.obuf = sbase + p.act_off + (l & 1) * p.act_buf_bytes;
                cx.bl = bias_s + L.bias_off;
                cx.act_lo = __float2half2_rn(L.act >= 1 ? 0.0f : -INFINITY);
                cx.act_hi = __float2half2_rn(L.act == 2 ? 6.0f : INFINITY);
                for (int c = 0; c < L.n_chunks && ok; c++) {
                    cx.ncols = chunk_cols(L, c);
                    cx.ch0 = c * L.chunk_n;
                    for (int b0 = 0; b0 < L.nb && ok; b0 += L.per_pass, pass_i++) {
                        const uint32_t half = pass_i & 1u;
                        ok = mbar_wait(&acc_full_bar[half], (pass_i >> 1) & 1u, abort_flag, p.status, 0x700 | (blockIdx.x << 12));
                        if (!ok) break;
                        DLF_TRACE_ACC(eacc, 0, emark);
                        tc_fence_after_sync();
                        cx.b0 = b0;
                        cx.nblk = min(L.per_pass, L.nb - b0);
                        cx.tmem_col = half * 256u;
                        if (mode == 0) epi_pass<0>(p, L, cx);
                        else if (mode == 1) epi_pass<1>(p, L, cx);
                        else if (mode == 2) epi_pass<2>(p, L, cx);
                        else epi_pass<3>(p, L, cx);
                        if (mode == 0 || mode == 3) fence_proxy_async_smem();  // UMMA reads these rows through the async proxy
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&acc_empty_bar[half]);
                        DLF_TRACE_ACC(eacc, 1 + mode, emark);
                    }
                }
                if (ok && !last && lane == 0) mbar_arrive(&act_ready_bar);
            }
            if (!ok) break;
            if (p.pool) {
                // ---- pooled copy-out from the staging buffer (coalesced 16-byte stores) -----------------
                epi_bar_sync();
                const uint8_t* obuf = sbase + p.act_off + ((p.n_layers - 1) & 1) * p.act_buf_bytes;
                const int c8n = p.cout_last / 8;
                const int oth = p.th / 2, otw = p.tw / 2;
                const int Ho = p.H / 2, Wo = p.W / 2;
                const int total = oth * otw * c8n;
                for (int i = et; i < total; i += 32 * kEpiWarps) {
                    const int g8 = i % c8n;
                    const int ox = (i / c8n) % otw, oy = i / (c8n * otw);
                    const int gy = tyi * oth + oy, gx = txi * otw + ox;
                    if (gy >= Ho || gx >= Wo) continue;
                    uint4 best = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int wq = 0; wq < 4; wq++) {
                        const int q = (p.halo + oy * 2 + (wq >> 1)) * p.pitch + p.halo + ox * 2 + (wq & 1);
                        const uint4 vv = *reinterpret_cast<const uint4*>(obuf + static_cast<size_t>(g8 >> 3) * p.plane_bytes +
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
                epi_bar_sync();
                DLF_TRACE_ACC(eacc, 5, emark);
            }
        }
        if (threadIdx.x == 0) DLF_TRACE_FLUSH_AT(p.status, eacc, 8);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) {
        if (abort_s) __nanosleep(20000);  // let copies in flight land before the CTA retires
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

int planes_of(int c) { return (c + 63) / 64; }
int pad16(int c) { return (c + 15) / 16 * 16; }

struct LayerGeom {
    int qs, range, nb, n_pad, n_chunks, chunk_n, slot, per_pass;
};

struct WeightBox {
    int tg, kg, rank4, bytes;
};

// Taps and K chunks per weight TMA box: as many as fit the target size, whole kernel rows first.
WeightBox weight_box(int cin, int cout, int k) {
    WeightBox w;
    const int n_pad = pad16(cout), chunk = n_pad > 256 ? 256 : n_pad;
    const int kchunks = planes_of(cin);
    w.rank4 = (cin % 64 == 0) ? 1 : 0;
    w.tg = 1;
    for (int t : {k * k, k}) {
        if (t * chunk * 128 <= kWeightOpBytes) { w.tg = t; break; }
    }
    w.kg = 1;
    if (w.rank4 && (w.tg == k * k || k == 1)) w.kg = std::max(1, std::min(kchunks, kWeightOpBytes / (w.tg * chunk * 128)));
    w.bytes = w.tg * w.kg * chunk * 128;
    return w;
}

LayerGeom layer_geom(int cout, int cum_pad, int rows, int pitch) {
    LayerGeom g;
    g.qs = cum_pad * pitch + cum_pad;
    g.range = (rows - 2 * cum_pad - 1) * pitch + (pitch - 2 * cum_pad);
    g.nb = (g.range + 127) / 128;
    g.n_pad = pad16(cout);
    g.n_chunks = (g.n_pad + 255) / 256;
    g.chunk_n = g.n_chunks == 1 ? g.n_pad : 256;
    g.slot = (std::min(g.chunk_n, g.n_pad) + 31) / 32 * 32;
    g.per_pass = 256 / g.slot;
    return g;
}

// Rows one activation plane must hold: the frame itself, plus what the last 128-row block of a
// layer may touch past it (its own rows when written, its farthest tap when read).
int rows_alloc_of(const ChainArgs& a, int rows, int pitch) {
    int need = rows * pitch, c = 0;
    for (int l = 0; l < a.n_layers; l++) {
        const int pad = a.k[l] / 2;
        c += pad;
        const LayerGeom g = layer_geom(a.cout[l], c, rows, pitch);
        need = std::max(need, g.qs + g.nb * 128 + pad * pitch + pad);
    }
    return (need + 7) / 8 * 8;
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
    return (k == 1 || k == 3) && cin % 8 == 0 && cout % 8 == 0 && cin >= 8 && cout >= 8 && cout <= 2048 && cin <= 1024;
}

// Picks the output tile from the SM count (Sec. IV-B: more cores -> smaller tiles -> more
// recomputed halo).  Among the tile shapes whose buffers fit in shared memory, takes the least
// estimated time = waves x per-tile time, the per-tile time being modelled in SM clocks from the
// UMMA issue rate (operand reads from shared memory vs. math), the epilogue and the input load.
ChainTiling chain_tc_tiling(const ChainArgs& a, int sm_count, int device_sms) {
    ChainTiling best{};
    best.ok = false;
    (void)device_sms;
    if (a.n_layers < 1 || a.n_layers > kMaxChain || sm_count < 1) return best;
    int halo = 0, bias_floats = 0, stage_n = 0;
    for (int l = 0; l < a.n_layers; l++) {
        if (!chain_tc_layer_supported(a.cin[l], a.cout[l], a.k[l])) return best;
        if (l > 0 && a.cin[l] != a.cout[l - 1]) return best;
        halo += a.k[l] / 2;
        bias_floats += pad16(a.cout[l]);
        stage_n = std::max(stage_n, weight_box(a.cin[l], a.cout[l], a.k[l]).bytes / 128);
    }
    if (bias_floats > kMaxBias) return best;
    const int L = a.n_layers;
    const int stage_bytes = stage_n * 128;
    const int in_planes = planes_of(a.cin[0]);
    int act_bufs = (L == 1) ? (a.pool ? 1 : 0) : ((L == 2 && !a.pool) ? 1 : 2);
    int act_planes = 0;
    for (int l = 0; l < L; l++)
        if (l < L - 1 || a.pool) act_planes = std::max(act_planes, planes_of(pad16(a.cout[l])));
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
    for (int th : cand_h)
        for (int tw : cand_w) {
            const int rows = th + 2 * halo, pitch = tw + 2 * halo;
            if (rows > 256 || pitch > 256) continue;
            const int rows_alloc = rows_alloc_of(a, rows, pitch);
            const size_t plane = static_cast<size_t>(rows_alloc) * 128;
            const size_t fixed = static_cast<size_t>(act_bufs) * act_planes * plane + static_cast<size_t>(bias_floats) * 4 + 1024;
            const int tiles_h = (a.H + th - 1) / th, tiles_w = (a.W + tw - 1) / tw;
            const long long n_tiles = static_cast<long long>(a.N) * tiles_h * tiles_w;
            if (n_tiles > 0x7fffffffLL) continue;
            const long long waves = (n_tiles + sm_count - 1) / sm_count;
            for (int in_bufs = 2; in_bufs >= 1; in_bufs--) {
                int stages = 3;
                auto total = [&](int st) { return fixed + static_cast<size_t>(in_bufs) * in_planes * plane + static_cast<size_t>(st) * stage_bytes; };
                while (stages > 2 && total(stages) > static_cast<size_t>(kMaxSmem)) stages--;
                if (total(stages) > static_cast<size_t>(kMaxSmem)) continue;
                double clk = 1500.0, useful = 0.0, computed = 0.0;
                int c = 0;
                for (int l = 0; l < L; l++) {
                    c += a.k[l] / 2;
                    const LayerGeom g = layer_geom(a.cout[l], c, rows, pitch);
                    const int ksteps = a.k[l] * a.k[l] * ((a.cin[l] + 15) / 16);
                    double mma = 0.0;
                    for (int ch = 0; ch < g.n_chunks; ch++) {
                        const int n = std::min(g.chunk_n, g.n_pad - ch * g.chunk_n);
                        // operand reads from shared memory: 4 KB of pixels (8 KB where the window straddles swizzle
                        // atoms: every tap of a 3x3 layer but the centre column's at a pitch that is a multiple of 8,
                        // else all but the centre tap) and n x 32 bytes of weights, at 128 bytes per clock
                        const double straddle = a.k[l] == 1 ? 0.0 : (pitch % 8 == 0 ? 6.0 / 9.0 : 8.0 / 9.0);
                        mma += static_cast<double>(g.nb) * ksteps * std::max(32.0 * (1.0 + straddle) + n / 4.0, n / 2.0);
                    }
                    const double epi = static_cast<double>(g.nb) * (g.n_pad / 32.0) * 220.0;
                    const int passes = g.n_chunks * ((g.nb + g.per_pass - 1) / g.per_pass);
                    clk += (passes > 1 ? std::max(mma, epi) + std::min(mma, epi) / passes : mma + epi) + 600.0;
                    computed += static_cast<double>(g.nb) * 128.0 * a.k[l] * a.k[l] * a.cin[l] * a.cout[l];
                    useful += static_cast<double>(std::min(th, a.H)) * std::min(tw, a.W) * a.k[l] * a.k[l] * a.cin[l] * a.cout[l];
                }
                const double load = static_cast<double>(rows) * pitch * in_planes * 128.0 / 48.0;
                clk = (in_bufs == 2) ? std::max(clk, load) : clk + load + 1500.0;
                const double cost = static_cast<double>(waves) * clk;
                if (!best.ok || cost < best.cost) {
                    best.th = th; best.tw = tw; best.halo = halo; best.pitch = pitch; best.rows = rows;
                    best.rows_alloc = rows_alloc;
                    best.tiles_h = tiles_h; best.tiles_w = tiles_w; best.n_tiles = static_cast<int>(n_tiles);
                    best.in_bufs = in_bufs; best.act_bufs = act_bufs; best.act_planes = act_planes;
                    best.stages = stages; best.stage_bytes = stage_bytes;
                    best.smem_bytes = total(stages);
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
    ChainParams p;
    std::memset(&p, 0, sizeof(p));
    p.n_layers = a.n_layers;
    p.N = a.N; p.H = a.H; p.W = a.W;
    p.th = t.th; p.tw = t.tw; p.halo = t.halo; p.pitch = t.pitch; p.rows = t.rows;
    p.tiles_h = t.tiles_h; p.tiles_w = t.tiles_w; p.n_tiles = t.n_tiles;
    p.plane_bytes = t.rows_alloc * 128;
    p.in_planes = planes_of(a.cin[0]);
    p.in_bufs = t.in_bufs;
    p.in_buf_bytes = p.in_planes * p.plane_bytes;
    p.act_off = p.in_bufs * p.in_buf_bytes;
    p.act_buf_bytes = t.act_planes * p.plane_bytes;
    p.ring_off = p.act_off + t.act_bufs * p.act_buf_bytes;
    p.stages = t.stages;
    p.stage_bytes = t.stage_bytes;
    p.bias_off = p.ring_off + p.stages * p.stage_bytes;
    int cum = 0, boff = 0;
    for (int l = 0; l < a.n_layers; l++) {
        ChainLayerP& L = p.L[l];
        L.cin = a.cin[l]; L.cout = a.cout[l]; L.k = a.k[l]; L.pad = a.k[l] / 2; L.act = a.act[l];
        L.kchunks = planes_of(a.cin[l]);
        L.ksteps_last = ((a.cin[l] - (L.kchunks - 1) * 64) + 15) / 16;
        cum += L.pad;
        const LayerGeom g = layer_geom(a.cout[l], cum, t.rows, t.pitch);
        L.qs = g.qs; L.range = g.range; L.nb = g.nb; L.n_pad = g.n_pad; L.n_chunks = g.n_chunks; L.chunk_n = g.chunk_n;
        L.slot = g.slot; L.per_pass = g.per_pass;
        L.bias_off = boff;
        boff += g.n_pad;
        L.bias = a.bias[l];
        const WeightBox wb = weight_box(a.cin[l], a.cout[l], a.k[l]);
        L.tg = wb.tg; L.kg = wb.kg; L.w_rank4 = wb.rank4;
        const uint64_t taps = static_cast<uint64_t>(a.k[l]) * a.k[l];
        const uint32_t box_n = static_cast<uint32_t>(std::min(g.chunk_n, g.n_pad));
        int rc;
        if (wb.rank4) {  // [cout][tap][cin] seen as (64 channels, cout, tap, cin / 64)
            const uint64_t dims[4] = {64, static_cast<uint64_t>(a.cout[l]), taps, static_cast<uint64_t>(a.cin[l] / 64)};
            const uint64_t strides[3] = {taps * a.cin[l] * 2, static_cast<uint64_t>(a.cin[l]) * 2, 128};
            const uint32_t box[4] = {64, box_n, static_cast<uint32_t>(wb.tg), static_cast<uint32_t>(wb.kg)};
            const uint32_t es[4] = {1, 1, 1, 1};
            rc = encode_tmap(&p.tmw[l], a.w[l], 4, dims, strides, box, es);
        } else {         // (cin, cout, tap): K chunks are addressed along dimension 0, zero-filled past cin
            const uint64_t dims[3] = {static_cast<uint64_t>(a.cin[l]), static_cast<uint64_t>(a.cout[l]), taps};
            const uint64_t strides[2] = {taps * a.cin[l] * 2, static_cast<uint64_t>(a.cin[l]) * 2};
            const uint32_t box[3] = {64, box_n, static_cast<uint32_t>(wb.tg)};
            const uint32_t es[3] = {1, 1, 1};
            rc = encode_tmap(&p.tmw[l], a.w[l], 3, dims, strides, box, es);
        }
        if (rc) return rc;
    }
    p.bias_floats = boff;
    p.pool = a.pool;
    p.cout_last = a.cout[a.n_layers - 1];
    p.res = static_cast<const __half*>(a.res);
    p.out = static_cast<__half*>(a.y);
    p.status = status_dev;
    {
        const uint64_t dims[4] = {static_cast<uint64_t>(a.cin[0]), static_cast<uint64_t>(a.W), static_cast<uint64_t>(a.H),
                                  static_cast<uint64_t>(a.N)};
        const uint64_t strides[3] = {static_cast<uint64_t>(a.cin[0]) * 2, static_cast<uint64_t>(a.W) * a.cin[0] * 2,
                                     static_cast<uint64_t>(a.H) * a.W * a.cin[0] * 2};
        const uint32_t box[4] = {64, static_cast<uint32_t>(t.pitch), static_cast<uint32_t>(t.rows), 1};
        const uint32_t es[4] = {1, 1, 1, 1};
        int rc = encode_tmap(&p.tmx, a.x, 4, dims, strides, box, es);
        if (rc) return rc;
    }
    const int grid = std::max(1, std::min(sm_count, t.n_tiles));
    const size_t smem = std::max<size_t>(t.smem_bytes, 120 * 1024);
#ifdef DLF_TRACE
    fprintf(stderr, "chain_tc: L=%d tile %dx%d frame %dx%d tiles %d grid %d in_bufs %d stages %d stage_bytes %d smem %zu red %.2f\n", a.n_layers,
            t.th, t.tw, t.rows, t.pitch, t.n_tiles, grid, t.in_bufs, t.stages, t.stage_bytes, t.smem_bytes, t.redundancy);
    for (int l = 0; l < a.n_layers; l++)
        fprintf(stderr, "  layer %d: %d->%d k%d nb %d chunks %d x %d per_pass %d tg %d kg %d\n", l, a.cin[l], a.cout[l], a.k[l], p.L[l].nb,
                p.L[l].n_chunks, p.L[l].chunk_n, p.L[l].per_pass, p.L[l].tg, p.L[l].kg);
#endif
    cudaError_t e = launch_kernel(chain_tc_kernel, grid, kThreads, smem, s, p);
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

int chain_tc_init() {
    static bool attr_set[kMaxDevices] = {};
    const int dev = current_device_slot();
    if (dev < 0) return DLF_E_UNSUPPORTED;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(chain_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e != cudaSuccess) return cuda_fail(e);
        attr_set[dev] = true;
    }
    return DLF_OK;
}

}  // namespace dlf
