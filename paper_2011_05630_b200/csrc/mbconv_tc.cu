// Fused inverted-residual block (MobileNetV2): 1x1 expansion (+bias, activation) -> depthwise 3x3,
// stride 1 or 2 (+bias, activation) -> 1x1 projection (+bias, optional residual, activation), as ONE
// kernel.  The expanded map (6x the block's input, the dominant HBM traffic of the unfused plan)
// never exists in memory: the hidden dimension is processed in chunks of 64 channels.  ALL THREE layers
// run on the tensor cores.  Per output tile and chunk:
//   1. expansion: D1[frame rows x 64] = X[frame rows x C_in] * W1[chunk]^T, the input frame (tile + 1-pixel
//      halo, TMA-loaded once per tile) staying in shared memory;
//   2. epilogue 1 (CUDA cores): bias, activation, fp16 rounding, zero outside the image (the depthwise layer's
//      padding) -> hidden frame H in shared memory, pixel-linear rows of 64 channels, 128-byte swizzled;
//   3. depthwise 3x3 as nine shifted products with DIAGONAL weight blocks: for tap (r, s) and each group of 16
//      channels, D[m, c] += H[m + shift(r, s), c'] * diag(w_tap)[c', c] is one M = 128, N = 16, K = 16 UMMA whose A
//      operand is the hidden frame itself, started (r * pitch + s) rows further on through the descriptor (no
//      copy, no im2col), and whose B operand is a 16 x 16 block holding the 16 channels' tap weights on its
//      diagonal (written once per chunk by the CUDA cores; the zeros around them never change).  Products with the
//      zeros add exactly 0, the nine real products are exact in fp32 and are summed in fp32: the layer's own sum
//      in another order.  The CUDA cores, which bounded the first version of this kernel (61 instructions per
//      hidden element for index arithmetic, conversions and fp32 multiply-adds), are left with two epilogues.
//      Stride 2: epilogue 1 writes the frame as four parity planes (even / odd row x even / odd column), so that
//      every tap of the stride-2 window is again a unit-stride shifted window in one of the planes;
//   4. epilogue 1.5: bias, activation, fp16 rounding of the depthwise sums -> dense tile Hd, the next operand;
//   5. projection: D2[tile rows x C_out] += Hd * W2[:, chunk]^T, accumulated in tensor memory across the chunks
//      (fp32, the same sum as the unchunked layer);
// then epilogue 2: bias, residual, activation, fp16 rounding.  Where shared memory has room the output
// tile is staged there and leaves through TMA stores issued by the input-producer warp, which also
// fetches the residual tile by TMA straight into that staging buffer a tile ahead (added in place);
// otherwise each thread stores and reads its own pixel's channels directly.  Every intermediate is
// rounded to fp16 exactly where the layer-by-layer execution rounds it.  Without an expansion layer
// (the network's first block; stride 1 only) steps 1-2 are skipped and the depthwise products read the input frame.
// The hidden frame and the depthwise accumulator are double-buffered where they fit: the tensor core multiplies chunk c
// while the CUDA cores round chunk c + 1's expansion and chunk c - 1's depthwise sums.
//
// Warps: 0-15 work (the epilogues), 16-18 UMMA issuers, 19 input producer, 20-21 weight producers.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstring>

#include "internal.h"
#include "ptx.cuh"

namespace dlf {

namespace {

// Trace build only: a timeline of CTA 0's issuer lane and first work thread (SM clock, event code) behind the status block.
#ifdef DLF_TRACE
#define DLF_TL(status, region, idx, code) do { if (blockIdx.x == 0 && idx < 250) { reinterpret_cast<volatile long long*>(status)[32 + (region) * 256 + idx] = (clock64() << 8) | (code); idx++; } } while (0)
#define DLF_TL_DECL(idx) int idx = 0
#else
#define DLF_TL(status, region, idx, code) do { } while (0)
#define DLF_TL_DECL(idx) do { } while (0)
#endif

constexpr int kWorkWarps = 16;
constexpr int kMmaWarp = kWorkWarps;
constexpr int kMma2Warp = kWorkWarps + 1;
constexpr int kMma3Warp = kWorkWarps + 2;
constexpr int kInWarp = kWorkWarps + 3;
constexpr int kW1Warp = kWorkWarps + 4;
constexpr int kW2Warp = kWorkWarps + 5;
constexpr int kThreads = 32 * (kWorkWarps + 6);
constexpr int kMaxSmem = 232448 - 1024;
constexpr int kMaxNb = 4;          // 128-row blocks of the frame / of the depthwise rows
constexpr int kDiagBytes = 9 * 2048;   // per chunk: nine strips of 16 rows x 128 bytes, four 16 x 16 blocks side by side in each

struct MbParams {
    CUtensorMap tmx, tmw1, tmw2, tmy, tmr;   // input frame, the two weight slabs, output tile, residual tile
    int N, H, W, Cin, hid, Cout, Ho, Wo, stride;
    int has_expand, act1, act2, act3;
    int th, tw, fh, fw, FR, nb1, nb2;   // output tile, input frame, frame rows, 128-row blocks of the expansion / projection
    int po, M, nbd;                     // depthwise rows: pitch (frame width; stride 2: width of a parity plane), count, 128-row blocks
    int PR;                             // stride 2: rows of one parity plane (a multiple of 8)
    int hbufs, ddbufs;                  // buffers of the hidden frame (with its diagonal blocks) / of the depthwise accumulator
    int tiles_h, tiles_w, n_tiles;
    int kin, chunks, n2_pad;            // 64-channel planes of the input, hidden chunks, C_out rounded up to 16
    int ksteps_in_last;
    int x_off, h_off, h_bytes, hd_off, diag_off, ring_off, stage_bytes, stages, bias_off;  // shared-memory byte offsets
    int so_off, so_planes;              // output staging buffer: byte offset, 64-channel planes (0: none, direct stores)
    int xplane, so_plane;               // bytes of one 64-channel plane of the input frame / of the staging buffer (rows rounded up to 8:
                                        // a UMMA reads 128 rows from a block's start, on into whatever follows; those accumulator rows are unused)
    int dd_col, d2_col;                 // first TMEM column of the depthwise / projection accumulators
    int w2_off, n_split, n_each;        // projection slab inside a ring stage; C_out > 256 is issued as two halves
    const __half* wd;
    const float *b1, *bd, *b2;
    const __half* res;
    __half* out;
    int* status;
};

// The four depthwise products of one tap (16-channel groups 0..3 of a chunk) in one statement: the frame window, the diagonal
// block and the accumulator columns advance by 32 bytes, 32 bytes and 16 columns per group.  (The issuing warp shares its
// scheduler with four work warps: every instruction saved on the way from one UMMA to the next shows in the kernel's time.)
__device__ __forceinline__ void umma_dw_x4(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t.reg .b32 ta, tb, td;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "mov.b64 da, {%1, %5};\n\tmov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
        "add.u32 ta, %1, 2;\n\tadd.u32 tb, %2, 2;\n\tadd.u32 td, %0, 16;\n\tmov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [td], da, db, %3, p;\n\t"
        "add.u32 ta, %1, 4;\n\tadd.u32 tb, %2, 4;\n\tadd.u32 td, %0, 32;\n\tmov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [td], da, db, %3, p;\n\t"
        "add.u32 ta, %1, 6;\n\tadd.u32 tb, %2, 6;\n\tadd.u32 td, %0, 48;\n\tmov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [td], da, db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHiSw128)
        : "memory");
}

__global__ void __launch_bounds__(kThreads, 1) mbconv_tc_kernel(const __grid_constant__ MbParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t x_full, x_empty, w1_full[4], w1_empty[4], w2_full[4], w2_empty[4], d1_full, d1_free, h_ready[2], h_free[2], dd_full[2], dd_free[2];
    __shared__ uint64_t hd_ready, hd_free, d2_full, d2_free, s_full, s_free;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sb = smem_raw + (base - smem_u32(smem_raw));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = &abort_s;
    float* bias_s = reinterpret_cast<float*>(sb + p.bias_off);  // b1[chunks * 64], bd[chunks * 64], b2[n2_pad]

    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(&x_full, 1);
        mbar_init(&x_empty, 1);
        for (int i = 0; i < p.stages; i++) {   // a ring stage holds a chunk's expansion slab and its projection slab, freed separately
            mbar_init(&w1_full[i], 1);
            mbar_init(&w1_empty[i], 1);
            mbar_init(&w2_full[i], 1);
            mbar_init(&w2_empty[i], 1);
        }
        mbar_init(&d1_full, 1);
        mbar_init(&d1_free, kWorkWarps);
        for (int i = 0; i < 2; i++) {
            mbar_init(&h_ready[i], kWorkWarps);
            mbar_init(&h_free[i], 1);
            mbar_init(&dd_full[i], 1);
            mbar_init(&dd_free[i], kWorkWarps);
        }
        mbar_init(&hd_ready, kWorkWarps);
        mbar_init(&hd_free, 1);
        mbar_init(&d2_full, 1);
        mbar_init(&d2_free, kWorkWarps);
        mbar_init(&s_full, kWorkWarps);
        mbar_init(&s_free, 1);
        fence_barrier_init();
        tma_prefetch_desc(&p.tmx);
        if (p.so_planes > 0) {
            tma_prefetch_desc(&p.tmy);
            if (p.res != nullptr) tma_prefetch_desc(&p.tmr);
        }
    }
    if (warp == kMmaWarp) {
        tmem_alloc(&tmem_base_s, 512);
        tmem_relinquish();
    }
    for (int i = threadIdx.x; i < p.chunks * 64; i += kThreads) {
        bias_s[i] = (p.has_expand && i < p.hid) ? __ldg(p.b1 + i) : 0.0f;
        bias_s[p.chunks * 64 + i] = i < p.hid ? __ldg(p.bd + i) : 0.0f;
    }
    for (int i = threadIdx.x; i < p.n2_pad; i += kThreads) bias_s[p.chunks * 128 + i] = i < p.Cout ? __ldg(p.b2 + i) : 0.0f;
    // the diagonal blocks' surroundings: zero for the whole kernel
    for (int i = threadIdx.x; i < p.hbufs * kDiagBytes / 16; i += kThreads) reinterpret_cast<uint4*>(sb + p.diag_off)[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();
    if (warp != kW1Warp && warp != kW2Warp) pdl_wait();  // the weight producers only read constants
    const uint32_t tmem_base = tmem_base_s;

    if (warp == kInWarp) {
        // ---- input producer: the tile's frame, one box per 64-channel plane; and, with a staging
        //      buffer, the finished tile out (TMA stores) and the next tile's residual in ------------------
        if (lane == 0) {
            const bool staged = p.so_planes > 0, has_res = p.res != nullptr;
            const uint32_t so_bytes = static_cast<uint32_t>(p.th * p.tw) * 128u;   // one plane's box
            auto fetch_residual = [&](int t) {
                const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h, n = t / (p.tiles_w * p.tiles_h);
                mbar_expect_tx(&s_free, static_cast<uint32_t>(p.so_planes) * so_bytes);
                for (int pl = 0; pl < p.so_planes; pl++)
                    tma_load_4d(sb + p.so_off + pl * p.so_plane, &p.tmr, &s_free, pl * 64, txi * p.tw, tyi * p.th, n);
            };
            // tile `ti_prev` is staged: send it off, wait until the buffer has been read, hand it back
            auto send_tile = [&](int t_prev, uint32_t ti_prev, int t_next) {
                if (!mbar_wait(&s_full, ti_prev & 1u, abort_flag, p.status, 0xB10 | (blockIdx.x << 12))) return false;
                const int txi = t_prev % p.tiles_w, tyi = (t_prev / p.tiles_w) % p.tiles_h, n = t_prev / (p.tiles_w * p.tiles_h);
                for (int pl = 0; pl < p.so_planes; pl++)
                    tma_store_4d(&p.tmy, sb + p.so_off + pl * p.so_plane, pl * 64, txi * p.tw, tyi * p.th, n);
                tma_store_commit();
                tma_store_wait_read();
                if (has_res) {
                    if (t_next < p.n_tiles) fetch_residual(t_next);
                } else {
                    mbar_arrive(&s_free);
                }
                return true;
            };
            if (staged && has_res && static_cast<int>(blockIdx.x) < p.n_tiles) fetch_residual(blockIdx.x);
            uint32_t ti = 0;
            int t_prev = -1;
            bool ok = true;
            for (int t = blockIdx.x; t < p.n_tiles; t += gridDim.x, ti++) {
                const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h, n = t / (p.tiles_w * p.tiles_h);
                ok = mbar_wait(&x_empty, (ti & 1u) ^ 1u, abort_flag, p.status, 0xB00 | (blockIdx.x << 12));
                if (!ok) break;
                mbar_expect_tx(&x_full, static_cast<uint32_t>(p.kin) * p.FR * 128u);
                for (int pl = 0; pl < p.kin; pl++)
                    tma_load_4d(sb + p.x_off + pl * p.xplane, &p.tmx, &x_full, pl * 64, txi * p.tw * p.stride - 1,
                                tyi * p.th * p.stride - 1, n);
                if (staged && t_prev >= 0) {
                    ok = send_tile(t_prev, ti - 1, t);
                    if (!ok) break;
                }
                t_prev = t;
            }
            if (staged && ok && t_prev >= 0) send_tile(t_prev, ti - 1, p.n_tiles);
        }
    } else if (warp == kW1Warp || warp == kW2Warp) {
        // ---- weight producers: per chunk the expansion slab [64 hidden][C_in] and the projection
        //      slab [C_out][64 hidden]; one ring stage holds both ---------------------------------------
        const bool w1 = warp == kW1Warp;
        if (lane == 0 && (!w1 || p.has_expand)) {
            int st = 0;          // ring position and phase as counters (no division on the way to a copy)
            uint32_t ph = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x)
                for (int hc = 0; hc < p.chunks; hc++) {
                    uint64_t* full = w1 ? &w1_full[st] : &w2_full[st];
                    ok = mbar_wait(w1 ? &w1_empty[st] : &w2_empty[st], ph ^ 1u, abort_flag, p.status, 0xC00 | (blockIdx.x << 12));
                    if (!ok) break;
                    uint8_t* dst = sb + p.ring_off + st * p.stage_bytes;
                    if (w1) {
                        mbar_expect_tx(full, static_cast<uint32_t>(p.kin) * 8192u);
                        for (int pl = 0; pl < p.kin; pl++) tma_load_3d(dst + pl * 8192, &p.tmw1, full, pl * 64, hc * 64, 0);
                    } else {
                        mbar_expect_tx(full, static_cast<uint32_t>(p.n2_pad) * 128u);
                        for (int j = 0; j < p.n_split; j++)
                            tma_load_3d(dst + p.w2_off + j * p.n_each * 128, &p.tmw2, full, hc * 64, j * p.n_each, 0);
                    }
                    if (++st == p.stages) { st = 0; ph ^= 1u; }
                }
        }
    } else if (warp == kMmaWarp) {
        // ---- first UMMA issuer: the depthwise products.  The whole warp walks the loops (warp-uniform descriptors), one
        //      elected lane issues.  Two issuing warps, because a warp's own instruction stream (waits, descriptor arithmetic,
        //      commits: hundreds of clocks per chunk) is not hidden behind the tensor core's queue, which is only a few
        //      instructions deep: while this warp is held inside the depthwise products, the other one gets the next
        //      expansion and the previous projection in between them.
        const uint32_t idescd = umma_idesc_f16(16);
        uint32_t ti = 0, cc = 0;  // tiles and chunks done so far (barrier phases)
        bool ok = true;
        DLF_TL_DECL(itl);
        DLF_TRACE_DECL(iacc, imark);  // CTA 0's first issuer: 1 hidden frame wait, 2 accumulator wait, 3 depthwise issue
        // offset of each tap's window in the hidden frame (stride 2: which parity plane, then the shift inside it), 16-byte units
        uint32_t tap_row[9];
#pragma unroll
        for (int t9 = 0; t9 < 9; t9++) {
            const int r = t9 / 3, s = t9 % 3;
            tap_row[t9] = 8u * (p.stride == 1 ? static_cast<uint32_t>(r * p.fw + s)
                                              : static_cast<uint32_t>(((r & 1) * 2 + (s & 1)) * p.PR + (r >> 1) * p.po + (s >> 1)));
        }
        const int last_hc = p.chunks - 1;
        int hc = 0;
        for (int t = blockIdx.x; t < p.n_tiles && ok; hc == last_hc ? (t += gridDim.x, ti++, hc = 0) : hc++, cc++) {
            const int jn = min(4, (p.hid - hc * 64) >> 4);   // 16-channel groups this chunk really has
            const uint32_t hb = cc & (p.hbufs - 1), db = cc & (p.ddbufs - 1);   // (one or two buffers each)
            // this chunk's hidden frame (and diagonal blocks) are written, the accumulator is drained
            ok = mbar_wait_warp(&h_ready[hb], (cc >> (p.hbufs - 1)) & 1u, abort_flag, p.status, 0xD80 | (blockIdx.x << 12));
            if (ok && !p.has_expand && hc == 0)   // (the depthwise products read the input frame itself)
                ok = mbar_wait_warp(&x_full, ti & 1u, abort_flag, p.status, 0xD00 | (blockIdx.x << 12));
            if (!ok) break;
            DLF_TRACE_ACC(iacc, 1, imark);
            if (lane == 0) DLF_TL(p.status, 0, itl, 1);
            if (cc >= static_cast<uint32_t>(p.ddbufs)) {
                ok = mbar_wait_warp(&dd_free[db], ((cc >> (p.ddbufs - 1)) - 1u) & 1u, abort_flag, p.status, 0xD90 | (blockIdx.x << 12));
                if (!ok) break;
            }
            DLF_TRACE_ACC(iacc, 2, imark);
            if (lane == 0) DLF_TL(p.status, 0, itl, 3);
            tc_fence_after_sync();
            const uint32_t h_lo = umma_desc_lo(p.has_expand ? base + p.h_off + hb * p.h_bytes : base + p.x_off + hc * p.xplane);
            const uint32_t g_lo = umma_desc_lo(base + p.diag_off + hb * kDiagBytes);
            if (elect_one()) {
                uint32_t hb_lo = h_lo, d_tmem = tmem_base + p.dd_col + db * p.nbd * 64u;
                for (int b = 0; b < p.nbd; b++, hb_lo += 1024u, d_tmem += 64u) {
#pragma unroll
                    for (int t9 = 0; t9 < 9; t9++) {
                        const uint32_t a_lo = hb_lo + tap_row[t9], b_lo = g_lo + t9 * 128u;
                        if (jn == 4) {
                            umma_dw_x4(d_tmem, a_lo, b_lo, idescd, t9 != 0);
                        } else {
                            for (int j = 0; j < jn; j++)
                                umma_f16_lo(d_tmem + 16u * j, a_lo + 2 * j, kDescHiSw128, b_lo + 2 * j, idescd, t9 != 0);
                        }
                    }
                }
                umma_commit(&dd_full[db]);
                umma_commit(&h_free[hb]);
                if (!p.has_expand && hc == last_hc) umma_commit(&x_empty);   // the frame itself was the operand
            }
            __syncwarp();
            DLF_TRACE_ACC(iacc, 3, imark);
            if (lane == 0) DLF_TL(p.status, 0, itl, 4);
        }
        if (lane == 0) DLF_TRACE_FLUSH_N(p.status, iacc, 16, 4);
    } else if (warp == kMma2Warp || warp == kMma3Warp) {
        // ---- second and third UMMA issuer: the expansions (one chunk ahead of the depthwise products) / the projections (one
        //      behind), each on its own warp so that neither waits for the other's events -------------------------------------
        const bool expander = warp == kMma2Warp;
        const uint32_t idesc1 = umma_idesc_f16(64), idesc2 = umma_idesc_f16(p.n_each);
        const int last_hc = p.chunks - 1;
        bool ok = true;
        DLF_TL_DECL(itl);
        int e_st = 0, j_st = 0;          // weight-ring positions and phases of the next expansion / projection, as counters
        uint32_t e_ph = 0, j_ph = 0;
        // D1 = X * W1[chunk]^T over the input planes; the weight stage is free again once these have read it
        auto issue_expand = [&](uint32_t c, bool first_of_tile, uint32_t tile_index, bool last_of_tile) -> bool {
            const int st = e_st;
            const uint32_t ph = e_ph;
            if (++e_st == p.stages) { e_st = 0; e_ph ^= 1u; }
            bool k = true;
            if (first_of_tile) k = mbar_wait_warp(&x_full, tile_index & 1u, abort_flag, p.status, 0xD00 | (blockIdx.x << 12));
            if (k) k = mbar_wait_warp(&w1_full[st], ph, abort_flag, p.status, 0xD10 | (blockIdx.x << 12));
            if (k && c > 0) k = mbar_wait_warp(&d1_free, (c - 1) & 1u, abort_flag, p.status, 0xD20 | (blockIdx.x << 12));
            if (!k) return false;
            tc_fence_after_sync();
            const uint32_t w_lo = umma_desc_lo(base + p.ring_off + st * p.stage_bytes), x_lo = umma_desc_lo(base + p.x_off);
            const uint32_t xplane16 = static_cast<uint32_t>(p.xplane) >> 4;
            if (elect_one()) {
                uint32_t b_lo = w_lo, xp_lo = x_lo;
                for (int pl = 0; pl < p.kin; pl++, b_lo += 512u, xp_lo += xplane16) {
                    const bool full = pl < p.kin - 1 || p.ksteps_in_last == 4;
                    uint32_t a_lo = xp_lo, d = tmem_base;
                    for (int b = 0; b < p.nb1; b++, a_lo += 1024u, d += 64u) {
                        if (full) {
                            umma_f16_x4(d, a_lo, b_lo, idesc1, pl != 0);
                        } else {
                            for (int ks = 0; ks < p.ksteps_in_last; ks++)
                                umma_f16_lo(d, a_lo + 2 * ks, kDescHiSw128, b_lo + 2 * ks, idesc1, (pl | ks) != 0);
                        }
                    }
                }
                umma_commit(&d1_full);
                umma_commit(&w1_empty[st]);
                if (last_of_tile) umma_commit(&x_empty);   // the frame is read by the expansions only
            }
            __syncwarp();
            if (lane == 0) DLF_TL(p.status, 0, itl, 2);
            return true;
        };
        // D2 += Hd * W2[:, chunk]^T once the chunk's depthwise tile is in shared memory
        auto issue_project = [&](uint32_t c, int hc_c, uint32_t ti_c) -> bool {
            const int st = j_st;
            const uint32_t ph = j_ph;
            if (++j_st == p.stages) { j_st = 0; j_ph ^= 1u; }
            const int jn = min(4, (p.hid - hc_c * 64) >> 4);
            bool k = mbar_wait_warp(&w2_full[st], ph, abort_flag, p.status, 0xD50 | (blockIdx.x << 12));
            if (k) k = mbar_wait_warp(&hd_ready, c & 1u, abort_flag, p.status, 0xD60 | (blockIdx.x << 12));
            if (k && hc_c == 0 && ti_c > 0) k = mbar_wait_warp(&d2_free, (ti_c - 1) & 1u, abort_flag, p.status, 0xD70 | (blockIdx.x << 12));
            if (!k) return false;
            if (lane == 0) DLF_TL(p.status, 0, itl, 5);
            tc_fence_after_sync();
            const uint32_t w_lo = umma_desc_lo(base + p.ring_off + st * p.stage_bytes + p.w2_off), hd_lo = umma_desc_lo(base + p.hd_off);
            if (elect_one()) {
                uint32_t b_lo = w_lo, d0 = tmem_base + p.d2_col;
                for (int j = 0; j < p.n_split; j++, b_lo += static_cast<uint32_t>(p.n_each) * 8u, d0 += p.n_each) {
                    uint32_t a_lo = hd_lo, d = d0;
                    for (int b = 0; b < p.nb2; b++, a_lo += 1024u, d += p.n2_pad) {
                        if (jn == 4) {
                            umma_f16_x4(d, a_lo, b_lo, idesc2, hc_c != 0);
                        } else {
                            for (int ks = 0; ks < jn; ks++)   // (channels past the hidden width are neither written nor read)
                                umma_f16_lo(d, a_lo + 2 * ks, kDescHiSw128, b_lo + 2 * ks, idesc2, (hc_c | ks) != 0);
                        }
                    }
                }
                umma_commit(&hd_free);
                umma_commit(&w2_empty[st]);
                if (hc_c == last_hc) umma_commit(&d2_full);
            }
            __syncwarp();
            if (lane == 0) DLF_TL(p.status, 0, itl, 6);
            return true;
        };
        // The chunks of all this CTA's tiles form one stream.  Chunk c + 1's expansion (of the next tile, behind a tile's last
        // chunk) is issued as soon as chunk c's first epilogue has read the expansion accumulator, chunk c's projection as soon
        // as its depthwise sums are rounded.
        int t = blockIdx.x, hc = 0;
        uint32_t ti = 0, cc = 0;
        if (expander && p.has_expand && t < p.n_tiles) ok = issue_expand(0, true, 0, last_hc == 0);
        while (t < p.n_tiles && ok) {
            const int t_next = hc == last_hc ? t + static_cast<int>(gridDim.x) : t, hc_next = hc == last_hc ? 0 : hc + 1;
            if (expander) {
                if (p.has_expand && t_next < p.n_tiles) ok = issue_expand(cc + 1, hc_next == 0, ti + 1, hc_next == last_hc);
            } else {
                ok = issue_project(cc, hc, ti);
            }
            cc++;
            if (hc == last_hc) ti++;
            t = t_next;
            hc = hc_next;
        }
    } else {
        // ---- work warps: epilogue 1 (+ the diagonal weight blocks), epilogue 1.5, epilogue 2 ---------------------------------
        const int wt = threadIdx.x;  // 0..511
        const int q = warp & 3, part = warp >> 2;   // TMEM lane quarter; which 16-column slice of every 64 columns
        const __half2 lo1 = __float2half2_rn(p.act1 >= 1 ? 0.0f : -INFINITY), hi1 = __float2half2_rn(p.act1 == 2 ? 6.0f : INFINITY);
        const __half2 lo2 = __float2half2_rn(p.act2 >= 1 ? 0.0f : -INFINITY), hi2 = __float2half2_rn(p.act2 == 2 ? 6.0f : INFINITY);
        const __half2 lo3 = __float2half2_rn(p.act3 >= 1 ? 0.0f : -INFINITY), hi3 = __float2half2_rn(p.act3 == 2 ? 6.0f : INFINITY);
        uint8_t* hdbuf = sb + p.hd_off;
        // This thread's rows never change: frame row r of expansion block b goes to row hrow[b] of the hidden frame (stride 2:
        // of its parity plane), frame position fyx[b]; depthwise row m of block b is output pixel orow[b] of the tile
        // (-1: a row between two tile rows or past the tile).
        int hrow[kMaxNb], fyx[kMaxNb], orow[kMaxNb];
#pragma unroll
        for (int b = 0; b < kMaxNb; b++) {
            const int r = b * 128 + q * 32 + lane;
            const int fy = r / p.fw, fx = r - fy * p.fw;
            fyx[b] = (fy << 16) | fx;
            hrow[b] = r >= p.FR ? -1 : (p.stride == 1 ? r : ((fy & 1) * 2 + (fx & 1)) * p.PR + (fy >> 1) * p.po + (fx >> 1));
            const int oy = r / p.po, ox = r - oy * p.po;
            orow[b] = (r < p.M && ox < p.tw) ? oy * p.tw + ox : -1;
        }
        uint32_t ti = 0, cc = 0;
        bool ok = true;
        DLF_TL_DECL(wtl);
        DLF_TRACE_DECL(wacc, wmark);  // CTA 0's thread 0: 0 frame-buffer wait, 1 diagonal blocks, 2 D1 wait, 3 epilogue 1, 4 depthwise wait, 5 Hd wait, 6 epilogue 1.5, 7 epilogue 2
        // the depthwise weights this thread puts on the diagonals, fetched one chunk ahead (chunk hc's: tap i / 64 of channel
        // hc * 64 + i % 64, for i = thread and thread + 512)
        __half dgv[2];
        auto fetch_diag = [&](int hc) {
#pragma unroll
            for (int k = 0; k < 2; k++) {
                const int i = wt + k * 32 * kWorkWarps;
                const int tp = i >> 6, ch = hc * 64 + (i & 63);
                dgv[k] = (i < 9 * 64 && ch < p.hid) ? __ldg(p.wd + static_cast<long long>(ch) * 9 + tp) : __float2half(0.0f);
            }
        };
        fetch_diag(0);
        // Epilogue 1 of chunk `c` (hidden chunk hc of the tile at frame origin (iy0, ix0)): the chunk's diagonal weight
        // blocks, then D1 -> hidden frame.
        auto epilogue1 = [&](uint32_t c, int hc, int iy0, int ix0) -> bool {
            const int jn = min(4, (p.hid - hc * 64) >> 4);
            const uint32_t hb = c & (p.hbufs - 1);
            if (c >= static_cast<uint32_t>(p.hbufs) &&
                !mbar_wait(&h_free[hb], ((c >> (p.hbufs - 1)) - 1u) & 1u, abort_flag, p.status, 0xE50 | (blockIdx.x << 12)))
                return false;
            DLF_TRACE_ACC(wacc, 0, wmark);
            if (threadIdx.x == 0) DLF_TL(p.status, 1, wtl, 10);
#pragma unroll
            for (int k = 0; k < 2; k++) {   // tap i / 64, channel i % 64 of the chunk (the values were fetched a chunk ahead)
                const int i = wt + k * 32 * kWorkWarps;
                const int tp = i >> 6, ch = i & 63, n = ch & 15;
                if (i < 9 * 64 && ch < jn * 16) {
                    const int unit = (2 * (ch >> 4) + (n >> 3)) ^ (n & 7);
                    *reinterpret_cast<__half*>(sb + p.diag_off + hb * kDiagBytes + tp * 2048 + n * 128 + (unit << 4) + (n & 7) * 2) = dgv[k];
                }
            }
            fetch_diag(hc + 1 == p.chunks ? 0 : hc + 1);
            DLF_TRACE_ACC(wacc, 1, wmark);
            if (p.has_expand) {
                if (!mbar_wait(&d1_full, c & 1u, abort_flag, p.status, 0xE10 | (blockIdx.x << 12))) return false;
                DLF_TRACE_ACC(wacc, 2, wmark);
                if (threadIdx.x == 0) DLF_TL(p.status, 1, wtl, 11);
                tc_fence_after_sync();
                if (part < jn) {
                    uint8_t* hbuf = sb + p.h_off + hb * p.h_bytes;
                    const float* bb = bias_s + hc * 64 + part * 16;
#pragma unroll
                    for (int b = 0; b < kMaxNb; b++) {
                        if (b >= p.nb1) break;
                        const int fy = fyx[b] >> 16, fx = fyx[b] & 0xffff;
                        const int gy = iy0 + fy, gx = ix0 + fx;
                        const bool in_img = gy >= 0 && gy < p.H && gx >= 0 && gx < p.W;
                        float v[16];
                        __syncwarp();
                        tmem_ld16(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + b * 64u + part * 16u, v);
                        const int hr = hrow[b];
                        if (hr >= 0) {
#pragma unroll
                            for (int g = 0; g < 2; g++) {
                                uint4 val = make_uint4(0u, 0u, 0u, 0u);
                                if (in_img) {
                                    const float4 ba = *reinterpret_cast<const float4*>(bb + g * 8), bc = *reinterpret_cast<const float4*>(bb + g * 8 + 4);
                                    val.x = pack_half2_clamp(v[g * 8 + 0] + ba.x, v[g * 8 + 1] + ba.y, lo1, hi1);
                                    val.y = pack_half2_clamp(v[g * 8 + 2] + ba.z, v[g * 8 + 3] + ba.w, lo1, hi1);
                                    val.z = pack_half2_clamp(v[g * 8 + 4] + bc.x, v[g * 8 + 5] + bc.y, lo1, hi1);
                                    val.w = pack_half2_clamp(v[g * 8 + 6] + bc.z, v[g * 8 + 7] + bc.w, lo1, hi1);
                                }
                                const int g8 = part * 2 + g;
                                *reinterpret_cast<uint4*>(hbuf + hr * 128 + ((g8 ^ (hr & 7)) << 4)) = val;
                            }
                        }
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&d1_free);
            }
            fence_proxy_async_smem();  // the depthwise UMMAs read the frame and the blocks through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(&h_ready[hb]);
            DLF_TRACE_ACC(wacc, 3, wmark);
            if (threadIdx.x == 0) DLF_TL(p.status, 1, wtl, 12);
            return true;
        };
        // Epilogue 1.5 of chunk `c`: depthwise sums -> Hd (dense tile rows, the projection's operand).
        auto epilogue15 = [&](uint32_t c, int hc) -> bool {
            const int jn = min(4, (p.hid - hc * 64) >> 4);
            const uint32_t db = c & (p.ddbufs - 1);
            if (!mbar_wait(&dd_full[db], (c >> (p.ddbufs - 1)) & 1u, abort_flag, p.status, 0xE60 | (blockIdx.x << 12))) return false;
            DLF_TRACE_ACC(wacc, 4, wmark);
            if (threadIdx.x == 0) DLF_TL(p.status, 1, wtl, 13);
            if (c > 0 && !mbar_wait(&hd_free, (c - 1) & 1u, abort_flag, p.status, 0xE20 | (blockIdx.x << 12))) return false;
            DLF_TRACE_ACC(wacc, 5, wmark);
            if (threadIdx.x == 0) DLF_TL(p.status, 1, wtl, 14);
            tc_fence_after_sync();
            if (part < jn) {
                const float* bb = bias_s + p.chunks * 64 + hc * 64 + part * 16;
#pragma unroll
                for (int b = 0; b < kMaxNb; b++) {
                    if (b >= p.nbd) break;
                    float v[16];
                    __syncwarp();
                    tmem_ld16(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + p.dd_col + (db * p.nbd + b) * 64u + part * 16u, v);
                    const int o = orow[b];
                    if (o >= 0) {
#pragma unroll
                        for (int g = 0; g < 2; g++) {
                            const float4 ba = *reinterpret_cast<const float4*>(bb + g * 8), bc = *reinterpret_cast<const float4*>(bb + g * 8 + 4);
                            uint4 val;
                            val.x = pack_half2_clamp(v[g * 8 + 0] + ba.x, v[g * 8 + 1] + ba.y, lo2, hi2);
                            val.y = pack_half2_clamp(v[g * 8 + 2] + ba.z, v[g * 8 + 3] + ba.w, lo2, hi2);
                            val.z = pack_half2_clamp(v[g * 8 + 4] + bc.x, v[g * 8 + 5] + bc.y, lo2, hi2);
                            val.w = pack_half2_clamp(v[g * 8 + 6] + bc.z, v[g * 8 + 7] + bc.w, lo2, hi2);
                            const int g8 = part * 2 + g;
                            *reinterpret_cast<uint4*>(hdbuf + o * 128 + ((g8 ^ (o & 7)) << 4)) = val;
                        }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&dd_free[db]);
            fence_proxy_async_smem();  // the projection UMMAs read Hd through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(&hd_ready);
            DLF_TRACE_ACC(wacc, 6, wmark);
            if (threadIdx.x == 0) DLF_TL(p.status, 1, wtl, 15);
            return true;
        };
        // Frame origin of a tile, then epilogue 1 of its chunk hc (stream position c).
        int e1_iy0 = 0, e1_ix0 = 0;   // (of the tile the first epilogues are at: the divisions are done once per tile)
        auto epilogue1_of = [&](uint32_t c, int t, int hc) -> bool {
            if (hc == 0) {
                const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h;
                e1_iy0 = tyi * p.th * p.stride - 1;
                e1_ix0 = txi * p.tw * p.stride - 1;
            }
            return epilogue1(c, hc, e1_iy0, e1_ix0);
        };
        // One stream of chunks over all this CTA's tiles: chunk c + 1's first epilogue (the next tile's, behind a tile's last
        // chunk) runs ahead of chunk c's second one - the tensor core multiplies chunk c meanwhile.
        if (static_cast<int>(blockIdx.x) < p.n_tiles) ok = epilogue1_of(0, blockIdx.x, 0);
        for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x, ti++) {
            const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h, n = t / (p.tiles_w * p.tiles_h);
            const int oy0 = tyi * p.th, ox0 = txi * p.tw;
            for (int hc = 0; hc < p.chunks && ok; hc++, cc++) {
                if (hc + 1 < p.chunks) ok = epilogue1_of(cc + 1, t, hc + 1);
                else if (t + static_cast<int>(gridDim.x) < p.n_tiles) ok = epilogue1_of(cc + 1, t + gridDim.x, 0);
                if (ok) ok = epilogue15(cc, hc);
            }
            if (!ok) break;
            // ---- epilogue 2: D2 -> global -------------------------------------------------------------------
            ok = mbar_wait(&d2_full, ti & 1u, abort_flag, p.status, 0xE30 | (blockIdx.x << 12));
            if (!ok) break;
            tc_fence_after_sync();
            if (threadIdx.x == 0) DLF_TL(p.status, 1, wtl, 16);
            const float* b2s = bias_s + p.chunks * 128;
            if (p.so_planes > 0) {
                // staged: the buffer is free again (first tile: at once) / holds this tile's residual
                ok = mbar_wait(&s_free, p.res != nullptr ? (ti & 1u) : ((ti & 1u) ^ 1u), abort_flag, p.status, 0xE40 | (blockIdx.x << 12));
                if (!ok) break;
                uint8_t* so = sb + p.so_off;
                const bool has_res = p.res != nullptr;
                for (int b = 0; b < p.nb2; b++) {
                    const int o = b * 128 + q * 32 + lane;
                    const bool live = o < p.th * p.tw;   // rows past the image are clipped by the TMA store
                    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + p.d2_col + b * p.n2_pad;
                    for (int c0 = part * 16; c0 < p.n2_pad; c0 += 64) {
                        float v[16];
                        __syncwarp();
                        tmem_ld16(taddr + c0, v);
                        if (!live) continue;
#pragma unroll
                        for (int g = 0; g < 2; g++) {
                            const int co = c0 + g * 8;
                            if (co >= p.Cout) break;
                            const int g8 = (co >> 3) & 7;
                            uint4* sp = reinterpret_cast<uint4*>(so + (co >> 6) * p.so_plane + o * 128 + ((g8 ^ (o & 7)) << 4));
                            const float4 ba = *reinterpret_cast<const float4*>(b2s + co), bc = *reinterpret_cast<const float4*>(b2s + co + 4);
                            float a[8] = {v[g * 8 + 0] + ba.x, v[g * 8 + 1] + ba.y, v[g * 8 + 2] + ba.z, v[g * 8 + 3] + ba.w,
                                          v[g * 8 + 4] + bc.x, v[g * 8 + 5] + bc.y, v[g * 8 + 6] + bc.z, v[g * 8 + 7] + bc.w};
                            if (has_res) {   // loaded into the staging buffer by TMA, zero outside the tensor
                                const uint4 rv = *sp;
                                const __half2* rh = reinterpret_cast<const __half2*>(&rv);
#pragma unroll
                                for (int e = 0; e < 4; e++) {
                                    const float2 f = __half22float2(rh[e]);
                                    a[2 * e] += f.x;
                                    a[2 * e + 1] += f.y;
                                }
                            }
                            uint4 val;
                            val.x = pack_half2_clamp(a[0], a[1], lo3, hi3);
                            val.y = pack_half2_clamp(a[2], a[3], lo3, hi3);
                            val.z = pack_half2_clamp(a[4], a[5], lo3, hi3);
                            val.w = pack_half2_clamp(a[6], a[7], lo3, hi3);
                            *sp = val;
                        }
                    }
                }
                fence_proxy_async_smem();  // the TMA store reads the staging buffer
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_full);
            } else
            for (int b = 0; b < p.nb2; b++) {
                const int o = b * 128 + q * 32 + lane;
                const int oy = o / p.tw, ox = o - oy * p.tw;
                const int gy = oy0 + oy, gx = ox0 + ox;
                const bool live = o < p.th * p.tw && gy < p.Ho && gx < p.Wo;
                const long long gpix = (static_cast<long long>(n) * p.Ho + gy) * p.Wo + gx;
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + p.d2_col + b * p.n2_pad;
                for (int c0 = part * 16; c0 < p.n2_pad; c0 += 64) {
                    float v[16];
                    __syncwarp();
                    tmem_ld16(taddr + c0, v);
                    if (!live) continue;
#pragma unroll
                    for (int g = 0; g < 2; g++) {
                        const int co = c0 + g * 8;
                        if (co >= p.Cout) break;
                        float a[8];
#pragma unroll
                        for (int e = 0; e < 8; e++) a[e] = v[g * 8 + e] + b2s[co + e];
                        if (p.res != nullptr) {
                            const uint4 rv = __ldg(reinterpret_cast<const uint4*>(p.res + gpix * p.Cout + co));
                            const __half2* rh = reinterpret_cast<const __half2*>(&rv);
#pragma unroll
                            for (int e = 0; e < 4; e++) {
                                const float2 f = __half22float2(rh[e]);
                                a[2 * e] += f.x;
                                a[2 * e + 1] += f.y;
                            }
                        }
                        uint4 val;
                        val.x = pack_half2_clamp(a[0], a[1], lo3, hi3);
                        val.y = pack_half2_clamp(a[2], a[3], lo3, hi3);
                        val.z = pack_half2_clamp(a[4], a[5], lo3, hi3);
                        val.w = pack_half2_clamp(a[6], a[7], lo3, hi3);
                        *reinterpret_cast<uint4*>(p.out + gpix * p.Cout + co) = val;
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&d2_free);
            DLF_TRACE_ACC(wacc, 7, wmark);
            if (threadIdx.x == 0) DLF_TL(p.status, 1, wtl, 17);
        }
        if (threadIdx.x == 0) DLF_TRACE_FLUSH_AT(p.status, wacc, 8);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) {
        if (abort_s) __nanosleep(20000);
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

int pad16(int c) { return (c + 15) / 16 * 16; }

// Shared-memory and tensor-memory layout of a tile choice; false if it does not fit.
struct MbLayout {
    int fh, fw, FR, nb1, nb2, po, M, nbd, PR, hbufs, ddbufs;
    int kin, chunks, n2;
    int x_off, h_off, h_bytes, hd_off, diag_off, ring_off, stage_bytes, stages, bias_off, so_off, so_planes, xplane, so_plane;
    int dd_col, d2_col;
    size_t smem;
};

bool mb_layout(const MbconvArgs& a, int th, int tw, MbLayout* L) {
    const int s = a.stride;
    L->fh = (th - 1) * s + 3; L->fw = (tw - 1) * s + 3;
    if (L->fh > 256 || L->fw > 256) return false;
    L->FR = L->fh * L->fw;
    L->nb1 = (L->FR + 127) / 128;
    L->nb2 = (th * tw + 127) / 128;
    L->po = s == 1 ? L->fw : tw + 1;
    L->M = (th - 1) * L->po + tw;
    L->nbd = (L->M + 127) / 128;
    L->PR = s == 1 ? 0 : ((th + 1) * (tw + 1) + 7) / 8 * 8;
    if (L->nb1 > kMaxNb || L->nbd > kMaxNb) return false;
    L->kin = (a.Cin + 63) / 64; L->chunks = (a.hid + 63) / 64; L->n2 = pad16(a.Cout);
    // hidden frame: frame rows (stride 2: four parity planes); the depthwise windows of the last rows read up to
    // 128 * nbd + 2 * pitch + 2 rows from a buffer's (plane's) start - whatever lies behind it in shared memory
    const int h_rows = s == 1 ? (L->FR + 7) / 8 * 8 : 4 * L->PR;
    L->h_bytes = h_rows * 128;
    L->xplane = (L->FR + 7) / 8 * 8 * 128;
    L->so_plane = (th * tw + 7) / 8 * 8 * 128;
    L->stage_bytes = L->kin * 8192 * (a.has_expand ? 1 : 0) + L->n2 * 128;
    const int d1_cols = a.has_expand ? L->nb1 * 64 : 0;
    const int bias_bytes = ((L->chunks * 128 + L->n2) * 4 + 1023) / 1024 * 1024;
    // the depthwise accumulator is double-buffered where tensor memory has the columns
    L->ddbufs = d1_cols + 2 * L->nbd * 64 + L->nb2 * L->n2 <= 512 ? 2 : 1;
    if (d1_cols + L->ddbufs * L->nbd * 64 + L->nb2 * L->n2 > 512) return false;
    // shared memory, by preference: three ring stages, two hidden frames, the output staging buffer; given up in that order
    for (int variant = 0; variant < 4; variant++) {
        L->stages = variant >= 1 ? 2 : 3;
        L->hbufs = (variant >= 2 && a.has_expand) ? 1 : 2;
        L->so_planes = variant >= 3 ? 0 : (a.Cout + 63) / 64;
        L->dd_col = d1_cols;
        L->d2_col = d1_cols + L->ddbufs * L->nbd * 64;
        L->x_off = 0;
        L->h_off = L->kin * L->xplane;
        L->hd_off = L->h_off + (a.has_expand ? L->hbufs * L->h_bytes : 0);
        L->diag_off = L->hd_off + L->so_plane;   // (Hd: the tile's rows, as one plane of the staging buffer)
        L->ring_off = (L->diag_off + L->hbufs * kDiagBytes + 1023) / 1024 * 1024;
        L->bias_off = (L->ring_off + L->stages * L->stage_bytes + 1023) / 1024 * 1024;
        L->so_off = L->bias_off + bias_bytes;
        // (+ slack: the last windows' reads past a frame, see above, stay inside the allocation)
        L->smem = static_cast<size_t>(L->so_off) + static_cast<size_t>(L->so_planes) * L->so_plane + 1024;
        {   // the windows' reads past the last frame (plane) must end inside the allocation
            const size_t last = a.has_expand ? static_cast<size_t>(L->h_off) + static_cast<size_t>(L->hbufs - 1) * L->h_bytes + static_cast<size_t>(3 * L->PR) * 128
                                             : static_cast<size_t>(L->x_off) + static_cast<size_t>(L->chunks - 1) * L->xplane;
            L->smem = std::max(L->smem, last + static_cast<size_t>(128 * L->nbd + 2 * L->po + 3) * 128 + 1024);
            L->smem = std::max(L->smem, static_cast<size_t>(L->h_off) + 128u * 128u * (L->nb1 + 1));   // (the expansion's reads past the last input plane)
        }
        if (L->smem <= static_cast<size_t>(kMaxSmem)) return true;
    }
    return false;
}

}  // namespace

bool mbconv_supported(const MbconvArgs& a) {
    if (a.Cin % 8 || a.hid % 16 || a.Cout % 8 || a.Cin > 256 || a.Cout > 512 || a.hid > 1024) return false;
    if (pad16(a.Cout) > 256 && pad16(a.Cout) % 32) return false;  // issued as two equal halves
    if (a.stride != 1 && a.stride != 2) return false;
    if (!a.has_expand && (a.hid != a.Cin || a.stride != 1)) return false;   // (the input frame is no set of parity planes)
    return a.N >= 1 && a.H >= 1 && a.W >= 1;
}

// Output tile of the fused block from the SM count: candidates whose buffers and accumulators fit,
// least (waves x per-tile work) in SM clocks.
MbconvTiling mbconv_tiling(const MbconvArgs& a, int sm_count) {
    MbconvTiling best{};
    best.ok = false;
    if (!mbconv_supported(a) || sm_count < 1) return best;
    const int Ho = (a.H + 2 - 3) / a.stride + 1, Wo = (a.W + 2 - 3) / a.stride + 1;
    double best_cost = -1.0;
    for (int th = 1; th <= 16; th++)
        for (int tw = 2; tw <= 32; tw++) {
            if (th > std::max(Ho, 2) || tw > std::max(Wo, 2)) continue;
            if (th * tw > 256) continue;
            MbLayout L;
            if (!mb_layout(a, th, tw, &L)) continue;
            const int tiles_h = (Ho + th - 1) / th, tiles_w = (Wo + tw - 1) / tw;
            const long long n_tiles = static_cast<long long>(a.N) * tiles_h * tiles_w;
            if (n_tiles > 0x7fffffffLL) continue;
            const long long waves = (n_tiles + sm_count - 1) / sm_count;
            // Per chunk (measured cycle accounts of one CTA): the tensor core runs nbd x 9 x (16-channel groups) depthwise
            // products of 40 clocks, the expansion and the projection; the work warps run the two epilogues, about 500 clocks
            // of dependent instructions per 128-row block and pass each; the two sides overlap but hand over to each other
            // four times per chunk (about 1500 clocks of waits).  Without both double buffers they alternate.
            const double jn = std::min(4.0, a.hid / 16.0 / L.chunks);
            const double tc = L.nbd * 9 * jn * 40.0 + (a.has_expand ? L.nb1 * L.kin * 4 * 50.0 : 0.0) + L.nb2 * 4 * std::max(48.0, L.n2 / 2.0);
            const double cu = (a.has_expand ? 500.0 + 500.0 * L.nb1 : 300.0) + 400.0 + 500.0 * L.nbd;
            const double per_chunk = (L.hbufs == 2 && L.ddbufs == 2) ? std::max(tc, cu) + 1500.0 : tc + cu + 1000.0;
            // epilogue 2: staged tiles leave by TMA; direct stores touch one cache line per thread and instruction
            const double epi2 = 1000.0 + L.nb2 * (L.n2 / 16.0) * (L.so_planes > 0 ? 400.0 : 1200.0);
            const double load = L.kin * L.FR * 128 / 64.0;   // the frame through the SM's fill port
            const double cost = static_cast<double>(waves) * (L.chunks * per_chunk + epi2 + std::max(0.0, load - L.chunks * per_chunk) + 1500.0);
            if (best_cost < 0 || cost < best_cost) {
                best_cost = cost;
                best.th = th; best.tw = tw; best.fh = L.fh; best.fw = L.fw; best.nb1 = L.nb1; best.nb2 = L.nb2;
                best.tiles_h = tiles_h; best.tiles_w = tiles_w; best.n_tiles = static_cast<int>(n_tiles);
                best.stages = L.stages; best.stage_bytes = L.stage_bytes;
                best.smem_bytes = L.smem;
                best.out_planes = L.so_planes;
                best.cost = cost;
                best.redundancy = static_cast<double>(L.FR) / (std::min(th, Ho) * a.stride * std::min(tw, Wo) * a.stride);
                best.ok = true;
            }
        }
    return best;
}

int mbconv_tc_init() {
    static bool attr_set[kMaxDevices] = {};
    const int dev = current_device_slot();
    if (dev < 0) return DLF_E_UNSUPPORTED;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(mbconv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e != cudaSuccess) return cuda_fail(e);
        attr_set[dev] = true;
    }
    return DLF_OK;
}

int launch_mbconv_tc(const MbconvArgs& a, const MbconvTiling& t, int sm_count, int* status_dev, cudaStream_t s) {
    if (!t.ok) return DLF_E_PLAN;
    int rc = mbconv_tc_init();
    if (rc) return rc;
    MbLayout L;
    if (!mbconv_supported(a) || !mb_layout(a, t.th, t.tw, &L)) return DLF_E_PLAN;
    MbParams p;
    std::memset(&p, 0, sizeof(p));
    p.N = a.N; p.H = a.H; p.W = a.W; p.Cin = a.Cin; p.hid = a.hid; p.Cout = a.Cout; p.stride = a.stride;
    p.Ho = (a.H + 2 - 3) / a.stride + 1; p.Wo = (a.W + 2 - 3) / a.stride + 1;
    p.has_expand = a.has_expand; p.act1 = a.act1; p.act2 = a.act2; p.act3 = a.act3;
    p.th = t.th; p.tw = t.tw; p.fh = L.fh; p.fw = L.fw; p.FR = L.FR; p.nb1 = L.nb1; p.nb2 = L.nb2;
    p.po = L.po; p.M = L.M; p.nbd = L.nbd; p.PR = L.PR; p.hbufs = L.hbufs; p.ddbufs = L.ddbufs;
    p.tiles_h = t.tiles_h; p.tiles_w = t.tiles_w; p.n_tiles = t.n_tiles;
    p.kin = L.kin; p.chunks = L.chunks; p.n2_pad = L.n2;
    p.ksteps_in_last = ((a.Cin - (p.kin - 1) * 64) + 15) / 16;
    p.x_off = L.x_off; p.h_off = L.h_off; p.h_bytes = L.h_bytes; p.hd_off = L.hd_off; p.diag_off = L.diag_off;
    p.ring_off = L.ring_off; p.stage_bytes = L.stage_bytes; p.stages = L.stages; p.bias_off = L.bias_off;
    p.so_off = L.so_off; p.so_planes = L.so_planes; p.xplane = L.xplane; p.so_plane = L.so_plane;
    p.dd_col = L.dd_col; p.d2_col = L.d2_col;
    p.w2_off = a.has_expand ? p.kin * 8192 : 0;
    p.n_split = p.n2_pad > 256 ? 2 : 1;
    p.n_each = p.n2_pad / p.n_split;
    p.wd = static_cast<const __half*>(a.wd); p.b1 = a.b1; p.bd = a.bd; p.b2 = a.b2;
    p.res = static_cast<const __half*>(a.res); p.out = static_cast<__half*>(a.y); p.status = status_dev;
    {
        const uint64_t dims[4] = {static_cast<uint64_t>(a.Cin), static_cast<uint64_t>(a.W), static_cast<uint64_t>(a.H), static_cast<uint64_t>(a.N)};
        const uint64_t strides[3] = {static_cast<uint64_t>(a.Cin) * 2, static_cast<uint64_t>(a.W) * a.Cin * 2,
                                     static_cast<uint64_t>(a.H) * a.W * a.Cin * 2};
        const uint32_t box[4] = {64, static_cast<uint32_t>(L.fw), static_cast<uint32_t>(L.fh), 1};
        const uint32_t es[4] = {1, 1, 1, 1};
        rc = encode_tmap(&p.tmx, a.x, 4, dims, strides, box, es);
        if (rc) return rc;
    }
    if (a.has_expand) {  // W1 [hid][C_in] seen as (C_in, hid, 1)
        const uint64_t dims[3] = {static_cast<uint64_t>(a.Cin), static_cast<uint64_t>(a.hid), 1};
        const uint64_t strides[2] = {static_cast<uint64_t>(a.Cin) * 2, static_cast<uint64_t>(a.hid) * a.Cin * 2};
        const uint32_t box[3] = {64, 64, 1};
        const uint32_t es[3] = {1, 1, 1};
        rc = encode_tmap(&p.tmw1, a.w1, 3, dims, strides, box, es);
        if (rc) return rc;
    }
    {  // W2 [C_out][hid] seen as (hid, C_out, 1)
        const uint64_t dims[3] = {static_cast<uint64_t>(a.hid), static_cast<uint64_t>(a.Cout), 1};
        const uint64_t strides[2] = {static_cast<uint64_t>(a.hid) * 2, static_cast<uint64_t>(a.Cout) * a.hid * 2};
        const uint32_t box[3] = {64, static_cast<uint32_t>(p.n_each), 1};
        const uint32_t es[3] = {1, 1, 1};
        rc = encode_tmap(&p.tmw2, a.w2, 3, dims, strides, box, es);
        if (rc) return rc;
    }
    if (p.so_planes > 0) {  // output (and residual) tile [C_out, Wo, Ho, N], one box per 64-channel plane
        const uint64_t dims[4] = {static_cast<uint64_t>(a.Cout), static_cast<uint64_t>(p.Wo), static_cast<uint64_t>(p.Ho), static_cast<uint64_t>(a.N)};
        const uint64_t strides[3] = {static_cast<uint64_t>(a.Cout) * 2, static_cast<uint64_t>(p.Wo) * a.Cout * 2,
                                     static_cast<uint64_t>(p.Ho) * p.Wo * a.Cout * 2};
        const uint32_t box[4] = {64, static_cast<uint32_t>(t.tw), static_cast<uint32_t>(t.th), 1};
        const uint32_t es[4] = {1, 1, 1, 1};
        rc = encode_tmap(&p.tmy, a.y, 4, dims, strides, box, es);
        if (rc) return rc;
        p.tmr = p.tmy;
        if (a.res) {
            rc = encode_tmap(&p.tmr, a.res, 4, dims, strides, box, es);
            if (rc) return rc;
        }
    }
    const int grid = std::max(1, std::min(sm_count, t.n_tiles));
    // (never two of these CTAs on an SM: each allocates all of tensor memory)
    const size_t smem = std::max<size_t>(L.smem, 120 * 1024);
    if (smem > static_cast<size_t>(kMaxSmem)) return DLF_E_PLAN;
    cudaError_t e = launch_kernel(mbconv_tc_kernel, grid, kThreads, smem, s, p);
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

}  // namespace dlf
