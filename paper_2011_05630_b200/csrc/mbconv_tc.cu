// Fused inverted-residual block (MobileNetV2): 1x1 expansion (+bias, activation) -> depthwise 3x3,
// stride 1 or 2 (+bias, activation) -> 1x1 projection (+bias, optional residual, activation), as ONE
// kernel.  The expanded map (6x the block's input, the dominant HBM traffic of the unfused plan)
// never exists in memory: the hidden dimension is processed in chunks of 64 channels.  Per output
// tile and chunk:
//   1. expansion on the tensor cores: D1[frame rows x 64] = X[frame rows x C_in] * W1[chunk]^T, the
//      input frame (tile + 1-pixel halo, TMA-loaded once per tile) staying in shared memory;
//   2. epilogue 1 (CUDA cores): bias, activation, fp16 rounding, zero outside the image (the
//      depthwise layer's padding) -> hidden tile H in shared memory;
//   3. depthwise 3x3 on the CUDA cores (exact per channel, so chunking the hidden dimension changes
//      nothing): nine 128-bit shared-memory reads per 8 channels, fp32 accumulate, bias, activation,
//      fp16 rounding -> tile Hd, laid out as the next GEMM's operand;
//   4. projection on the tensor cores: D2[tile rows x C_out] += Hd * W2[:, chunk]^T, accumulated in
//      tensor memory across the chunks (fp32, the same sum as the unchunked layer);
// then epilogue 2: bias, residual, activation, fp16 rounding.  Where shared memory has room the output
// tile is staged there and leaves through TMA stores issued by the input-producer warp, which also
// fetches the residual tile by TMA straight into that staging buffer a tile ahead (added in place);
// otherwise each thread stores and reads its own pixel's channels directly.  Every intermediate is
// rounded to fp16 exactly where the layer-by-layer execution rounds it.  Without an expansion layer
// (the network's first block) steps 1-2 are skipped and the depthwise layer reads the input frame.
//
// Warps: 0-15 work (epilogues and depthwise; a thread keeps FOUR channels' depthwise weights in registers so that
// sixteen warps fit the register file), 16 UMMA issuer, 17 input producer, 18-19 weight producers.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstring>

#include "internal.h"
#include "ptx.cuh"

namespace dlf {

namespace {

constexpr int kWorkWarps = 16;   // with eight the CUDA-core phases ran at 0.4 instructions per scheduler cycle (measured)
constexpr int kMmaWarp = kWorkWarps;
constexpr int kInWarp = kWorkWarps + 1;
constexpr int kW1Warp = kWorkWarps + 2;
constexpr int kW2Warp = kWorkWarps + 3;
constexpr int kThreads = 32 * (kWorkWarps + 4);
constexpr int kMaxSmem = 232448 - 1024;
constexpr int kPlane = 128 * 128;  // 128 rows x 64 channels

struct MbParams {
    CUtensorMap tmx, tmw1, tmw2, tmy, tmr;   // input frame, the two weight slabs, output tile, residual tile
    int N, H, W, Cin, hid, Cout, Ho, Wo, stride;
    int has_expand, act1, act2, act3;
    int th, tw, fh, fw, FR, nb1, nb2;   // output tile, input frame, frame rows, 128-row blocks of the two GEMMs
    int tiles_h, tiles_w, n_tiles;
    int kin, chunks, n2_pad;            // 64-channel planes of the input, hidden chunks, C_out rounded up to 16
    int ksteps_in_last;
    int x_off, h_off, hd_off, ring_off, stage_bytes, stages, dw_off, bias_off;  // shared-memory byte offsets
    int so_off, so_planes;              // output staging buffer: byte offset, 64-channel planes (0: none, direct stores)
    int d2_col;                         // first TMEM column of the projection accumulator
    int w2_off, n_split, n_each;        // projection slab inside a ring stage; C_out > 256 is issued as two halves
    const __half* wd;
    const float *b1, *bd, *b2;
    const __half* res;
    __half* out;
    int* status;
};

__device__ __forceinline__ void work_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(32 * kWorkWarps) : "memory"); }


// Depthwise 3x3 of one 4-channel group (8 bytes of a pixel's 128-byte row; g4 = 0..15) for two horizontally
// adjacent output pixels: the input vectors the two windows share are read from shared memory and converted once.
template <int STRIDE>
__device__ __forceinline__ void dw_pair(const uint8_t* hsrc, uint8_t* hdbuf, int fw, int tw, int g4, int oy, int ox, bool second,
                                        const float (&wreg)[9][4], const float (&breg)[4], __half2 lo, __half2 hi) {
    constexpr int kCols = STRIDE + 3;  // input columns the two windows cover
    const int g8 = g4 >> 1, sub = (g4 & 1) * 8;
    float acc[2][4];
#pragma unroll
    for (int e = 0; e < 4; e++) acc[0][e] = acc[1][e] = 0.0f;
#pragma unroll
    for (int r = 0; r < 3; r++) {
        const int q0 = (oy * STRIDE + r) * fw + ox * STRIDE;
        uint2 xv[kCols];
#pragma unroll
        for (int c = 0; c < kCols; c++) xv[c] = *reinterpret_cast<const uint2*>(hsrc + (q0 + c) * 128 + ((g8 ^ ((q0 + c) & 7)) << 4) + sub);
#pragma unroll
        for (int c = 0; c < kCols; c++) {
            const __half2* xh = reinterpret_cast<const __half2*>(&xv[c]);
            const float2 f0 = __half22float2(xh[0]), f1 = __half22float2(xh[1]);
            const float xf[4] = {f0.x, f0.y, f1.x, f1.y};
            if (c < 3) {
#pragma unroll
                for (int e = 0; e < 4; e++) acc[0][e] = fmaf(xf[e], wreg[r * 3 + c][e], acc[0][e]);
            }
            if (c >= STRIDE) {
#pragma unroll
                for (int e = 0; e < 4; e++) acc[1][e] = fmaf(xf[e], wreg[r * 3 + c - STRIDE][e], acc[1][e]);
            }
        }
    }
#pragma unroll
    for (int k = 0; k < 2; k++) {
        if (k == 1 && !second) break;
        const int o = oy * tw + ox + k;
        uint2 val;
        val.x = pack_half2_clamp(acc[k][0] + breg[0], acc[k][1] + breg[1], lo, hi);
        val.y = pack_half2_clamp(acc[k][2] + breg[2], acc[k][3] + breg[3], lo, hi);
        *reinterpret_cast<uint2*>(hdbuf + o * 128 + ((g8 ^ (o & 7)) << 4) + sub) = val;
    }
}

__global__ void __launch_bounds__(kThreads, 1) mbconv_tc_kernel(const __grid_constant__ MbParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t x_full, x_empty, w_full[4], w_empty[4], d1_full, d1_free, hd_ready, hd_free, d2_full, d2_free, s_full, s_free;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sb = smem_raw + (base - smem_u32(smem_raw));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = &abort_s;
    float* bias_s = reinterpret_cast<float*>(sb + p.bias_off);  // b1[chunks * 64] then b2[n2_pad]

    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(&x_full, 1);
        mbar_init(&x_empty, p.has_expand ? 1 : kWorkWarps);
        for (int i = 0; i < p.stages; i++) {
            mbar_init(&w_full[i], p.has_expand ? 2 : 1);
            mbar_init(&w_empty[i], 1);
        }
        mbar_init(&d1_full, 1);
        mbar_init(&d1_free, kWorkWarps);
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
    for (int i = threadIdx.x; i < p.chunks * 64; i += kThreads) bias_s[i] = (p.has_expand && i < p.hid) ? __ldg(p.b1 + i) : 0.0f;
    for (int i = threadIdx.x; i < p.n2_pad; i += kThreads) bias_s[p.chunks * 64 + i] = i < p.Cout ? __ldg(p.b2 + i) : 0.0f;
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
                    tma_load_4d(sb + p.so_off + pl * p.nb2 * kPlane, &p.tmr, &s_free, pl * 64, txi * p.tw, tyi * p.th, n);
            };
            // tile `ti_prev` is staged: send it off, wait until the buffer has been read, hand it back
            auto send_tile = [&](int t_prev, uint32_t ti_prev, int t_next) {
                if (!mbar_wait(&s_full, ti_prev & 1u, abort_flag, p.status, 0xB10 | (blockIdx.x << 12))) return false;
                const int txi = t_prev % p.tiles_w, tyi = (t_prev / p.tiles_w) % p.tiles_h, n = t_prev / (p.tiles_w * p.tiles_h);
                for (int pl = 0; pl < p.so_planes; pl++)
                    tma_store_4d(&p.tmy, sb + p.so_off + pl * p.nb2 * kPlane, pl * 64, txi * p.tw, tyi * p.th, n);
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
                    tma_load_4d(sb + p.x_off + pl * p.nb1 * kPlane, &p.tmx, &x_full, pl * 64, txi * p.tw * p.stride - 1,
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
        if (lane == 0 && (warp == kW2Warp || p.has_expand)) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x)
                for (int hc = 0; hc < p.chunks; hc++, it++) {
                    const int st = it % p.stages;
                    ok = mbar_wait(&w_empty[st], ((it / p.stages) & 1u) ^ 1u, abort_flag, p.status, 0xC00 | (blockIdx.x << 12));
                    if (!ok) break;
                    uint8_t* dst = sb + p.ring_off + st * p.stage_bytes;
                    if (warp == kW1Warp) {
                        mbar_expect_tx(&w_full[st], static_cast<uint32_t>(p.kin) * 8192u);
                        for (int pl = 0; pl < p.kin; pl++) tma_load_3d(dst + pl * 8192, &p.tmw1, &w_full[st], pl * 64, hc * 64, 0);
                    } else {
                        mbar_expect_tx(&w_full[st], static_cast<uint32_t>(p.n2_pad) * 128u);
                        for (int j = 0; j < p.n_split; j++)
                            tma_load_3d(dst + p.w2_off + j * p.n_each * 128, &p.tmw2, &w_full[st], hc * 64, j * p.n_each, 0);
                    }
                }
        }
    } else if (warp == kMmaWarp) {
        // ---- UMMA issuer -------------------------------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc1 = umma_idesc_f16(64), idesc2 = umma_idesc_f16(p.n_each);
            uint32_t ti = 0, cc = 0;  // tiles and chunks done so far (barrier phases)
            bool ok = true;
            auto issue_expand = [&](uint32_t chunk_index) {
                // D1 = X * W1[chunk]^T over the input planes
                const int st = chunk_index % p.stages;
                const uint32_t wsm = base + p.ring_off + st * p.stage_bytes;
                for (int pl = 0; pl < p.kin; pl++) {
                    const int ksteps = (pl == p.kin - 1) ? p.ksteps_in_last : 4;
                    const uint32_t b_lo = umma_desc_lo(wsm + pl * 8192);
                    for (int b = 0; b < p.nb1; b++) {
                        const uint32_t a_lo = umma_desc_lo(base + p.x_off + (pl * p.nb1 + b) * kPlane);
                        for (int ks = 0; ks < ksteps; ks++)
                            umma_f16_lo(tmem_base + b * 64u, a_lo + 2 * ks, kDescHiSw128, b_lo + 2 * ks, idesc1, (pl | ks) != 0);
                    }
                }
                umma_commit(&d1_full);
            };
            for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x, ti++) {
                ok = mbar_wait(&x_full, ti & 1u, abort_flag, p.status, 0xD00 | (blockIdx.x << 12));
                if (!ok) break;
                tc_fence_after_sync();
                if (p.has_expand) {
                    ok = mbar_wait(&w_full[cc % p.stages], (cc / p.stages) & 1u, abort_flag, p.status, 0xD10 | (blockIdx.x << 12));
                    if (ok && cc > 0) ok = mbar_wait(&d1_free, (cc - 1) & 1u, abort_flag, p.status, 0xD20 | (blockIdx.x << 12));
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue_expand(cc);
                }
                for (int hc = 0; hc < p.chunks && ok; hc++, cc++) {
                    if (p.has_expand && hc + 1 < p.chunks) {
                        // the next chunk's expansion overlaps this chunk's depthwise step
                        ok = mbar_wait(&w_full[(cc + 1) % p.stages], ((cc + 1) / p.stages) & 1u, abort_flag, p.status, 0xD30 | (blockIdx.x << 12));
                        if (ok) ok = mbar_wait(&d1_free, cc & 1u, abort_flag, p.status, 0xD40 | (blockIdx.x << 12));
                        if (!ok) break;
                        tc_fence_after_sync();
                        issue_expand(cc + 1);
                    } else if (!p.has_expand) {
                        ok = mbar_wait(&w_full[cc % p.stages], (cc / p.stages) & 1u, abort_flag, p.status, 0xD50 | (blockIdx.x << 12));
                        if (!ok) break;
                    }
                    if (p.has_expand && hc + 1 == p.chunks) umma_commit(&x_empty);  // the frame is read by the expansions only
                    // projection of this chunk once its depthwise tile is in shared memory
                    ok = mbar_wait(&hd_ready, cc & 1u, abort_flag, p.status, 0xD60 | (blockIdx.x << 12));
                    if (ok && hc == 0 && ti > 0) ok = mbar_wait(&d2_free, (ti - 1) & 1u, abort_flag, p.status, 0xD70 | (blockIdx.x << 12));
                    if (!ok) break;
                    tc_fence_after_sync();
                    const int st = cc % p.stages;
                    for (int j = 0; j < p.n_split; j++) {
                        const uint32_t b_lo = umma_desc_lo(base + p.ring_off + st * p.stage_bytes + p.w2_off + j * p.n_each * 128);
                        for (int b = 0; b < p.nb2; b++) {
                            const uint32_t a_lo = umma_desc_lo(base + p.hd_off + b * kPlane);
                            for (int ks = 0; ks < 4; ks++)
                                umma_f16_lo(tmem_base + p.d2_col + b * p.n2_pad + j * p.n_each, a_lo + 2 * ks, kDescHiSw128, b_lo + 2 * ks,
                                            idesc2, (hc | ks) != 0);
                        }
                    }
                    umma_commit(&hd_free);
                    umma_commit(&w_empty[st]);
                    if (hc + 1 == p.chunks) umma_commit(&d2_full);
                }
            }
        }
    } else {
        // ---- work warps: epilogue 1, depthwise, epilogue 2 ---------------------------------------------------
        const int wt = threadIdx.x;  // 0..255
        const int q = warp & 3, part = warp >> 2;   // TMEM lane quarter; which 16-column slice of every 64 columns
        const __half2 lo1 = __float2half2_rn(p.act1 >= 1 ? 0.0f : -INFINITY), hi1 = __float2half2_rn(p.act1 == 2 ? 6.0f : INFINITY);
        const __half2 lo2 = __float2half2_rn(p.act2 >= 1 ? 0.0f : -INFINITY), hi2 = __float2half2_rn(p.act2 == 2 ? 6.0f : INFINITY);
        const __half2 lo3 = __float2half2_rn(p.act3 >= 1 ? 0.0f : -INFINITY), hi3 = __float2half2_rn(p.act3 == 2 ? 6.0f : INFINITY);
        uint8_t* hbuf = sb + (p.has_expand ? p.h_off : p.x_off);
        uint8_t* hdbuf = sb + p.hd_off;
        uint32_t ti = 0, cc = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x, ti++) {
            const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h, n = t / (p.tiles_w * p.tiles_h);
            const int oy0 = tyi * p.th, ox0 = txi * p.tw;
            const int iy0 = oy0 * p.stride - 1, ix0 = ox0 * p.stride - 1;
            if (!p.has_expand) {
                ok = mbar_wait(&x_full, ti & 1u, abort_flag, p.status, 0xE00 | (blockIdx.x << 12));
                if (!ok) break;
            }
            for (int hc = 0; hc < p.chunks && ok; hc++, cc++) {
                // this thread's depthwise weights and bias: it keeps one 4-channel group of the chunk for all
                // its pixels (512 threads, 16 groups: the group index is the thread index modulo 16)
                const int groups = min(16, (p.hid - hc * 64 + 3) >> 2);  // 4-channel groups this chunk really has
                float wreg[9][4], breg[4];
                {
                    const int ch0 = hc * 64 + (wt & 15) * 4;
                    if ((wt & 15) < groups) {
                        __align__(8) __half wv[36];   // 4 channels x 9 taps, consecutive in memory from ch0 * 9
                        const uint2* wp2 = reinterpret_cast<const uint2*>(p.wd + static_cast<long long>(ch0) * 9);
#pragma unroll
                        for (int k = 0; k < 9; k++) reinterpret_cast<uint2*>(wv)[k] = __ldg(wp2 + k);
#pragma unroll
                        for (int e = 0; e < 4; e++) {
                            breg[e] = __ldg(p.bd + ch0 + e);
#pragma unroll
                            for (int tp = 0; tp < 9; tp++) wreg[tp][e] = __half2float(wv[e * 9 + tp]);
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; e++) {
                            breg[e] = 0.0f;
#pragma unroll
                            for (int tp = 0; tp < 9; tp++) wreg[tp][e] = 0.0f;
                        }
                    }
                }
                if (p.has_expand) {
                    // ---- epilogue 1: D1 -> H (fp16, zero outside the image) ------------------------------
                    ok = mbar_wait(&d1_full, cc & 1u, abort_flag, p.status, 0xE10 | (blockIdx.x << 12));
                    if (!ok) break;
                    tc_fence_after_sync();
                    for (int b = 0; b < p.nb1; b++) {
                        const int r = b * 128 + q * 32 + lane;
                        const int fy = r / p.fw, fx = r - fy * p.fw;
                        const int gy = iy0 + fy, gx = ix0 + fx;
                        const bool in_img = r < p.FR && gy >= 0 && gy < p.H && gx >= 0 && gx < p.W;
                        float v[16];
                        __syncwarp();
                        tmem_ld16(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + b * 64u + part * 16u, v);
                        if (r < p.FR) {
                            const float* bb = bias_s + hc * 64 + part * 16;
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
                                *reinterpret_cast<uint4*>(hbuf + r * 128 + ((g8 ^ (r & 7)) << 4)) = val;
                            }
                        }
                    }
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&d1_free);
                }
                work_bar_sync();  // H complete
                if (cc > 0) {
                    ok = mbar_wait(&hd_free, (cc - 1) & 1u, abort_flag, p.status, 0xE20 | (blockIdx.x << 12));
                    if (!ok) break;
                }
                // ---- depthwise 3x3: H -> Hd ---------------------------------------------------------------
                const uint8_t* hsrc = hbuf + (p.has_expand ? 0 : hc * p.nb1 * kPlane);
                const int pairs_w = (p.tw + 1) >> 1;
                for (int item = wt; item < p.th * pairs_w * 16; item += 32 * kWorkWarps) {
                    const int g4 = item & 15, pr = item >> 4;
                    const int oy = pr / pairs_w, ox = (pr - oy * pairs_w) * 2;
                    const bool second = ox + 1 < p.tw;
                    if (g4 < groups) {
                        // the second window of a last, odd pair reads columns past the frame row: still inside the
                        // buffer (next row or slack), and its result is not stored
                        if (p.stride == 1) dw_pair<1>(hsrc, hdbuf, p.fw, p.tw, g4, oy, ox, second, wreg, breg, lo2, hi2);
                        else dw_pair<2>(hsrc, hdbuf, p.fw, p.tw, g4, oy, ox, second, wreg, breg, lo2, hi2);
                    } else {  // channel groups the chunk does not have: zero operand columns
                        const int o = oy * p.tw + ox, g8 = g4 >> 1, sub = (g4 & 1) * 8;
                        *reinterpret_cast<uint2*>(hdbuf + o * 128 + ((g8 ^ (o & 7)) << 4) + sub) = make_uint2(0u, 0u);
                        if (second) *reinterpret_cast<uint2*>(hdbuf + (o + 1) * 128 + ((g8 ^ ((o + 1) & 7)) << 4) + sub) = make_uint2(0u, 0u);
                    }
                }
                fence_proxy_async_smem();  // the projection UMMAs read Hd through the async proxy
                __syncwarp();
                if (lane == 0) mbar_arrive(&hd_ready);
                if (!p.has_expand && hc + 1 == p.chunks && lane == 0) mbar_arrive(&x_empty);
                work_bar_sync();  // nobody still reads H when the next chunk overwrites it
            }
            if (!ok) break;
            // ---- epilogue 2: D2 -> global -------------------------------------------------------------------
            ok = mbar_wait(&d2_full, ti & 1u, abort_flag, p.status, 0xE30 | (blockIdx.x << 12));
            if (!ok) break;
            tc_fence_after_sync();
            const float* b2s = bias_s + p.chunks * 64;
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
                            uint4* sp = reinterpret_cast<uint4*>(so + (co >> 6) * p.nb2 * kPlane + o * 128 + ((g8 ^ (o & 7)) << 4));
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
        }
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

}  // namespace

bool mbconv_supported(const MbconvArgs& a) {
    if (a.Cin % 8 || a.hid % 16 || a.Cout % 8 || a.Cin > 256 || a.Cout > 512 || a.hid > 1024) return false;
    if (pad16(a.Cout) > 256 && pad16(a.Cout) % 32) return false;  // issued as two equal halves
    if (a.stride != 1 && a.stride != 2) return false;
    if (!a.has_expand && a.hid != a.Cin) return false;
    return a.N >= 1 && a.H >= 1 && a.W >= 1;
}

// Output tile of the fused block from the SM count: candidates whose buffers and accumulators fit,
// least (waves x per-tile work).
MbconvTiling mbconv_tiling(const MbconvArgs& a, int sm_count) {
    MbconvTiling best{};
    best.ok = false;
    if (!mbconv_supported(a) || sm_count < 1) return best;
    const int Ho = (a.H + 2 - 3) / a.stride + 1, Wo = (a.W + 2 - 3) / a.stride + 1;
    const int kin = (a.Cin + 63) / 64, chunks = (a.hid + 63) / 64, n2 = pad16(a.Cout);
    static const int cand[] = {2, 4, 7, 8, 14, 16};
    double best_cost = -1.0;
    for (int th : cand)
        for (int tw : cand) {
            if (th > std::max(Ho, 2) * 2 || tw > std::max(Wo, 2) * 2) continue;
            const int fh = (th - 1) * a.stride + 3, fw = (tw - 1) * a.stride + 3;
            if (fh > 256 || fw > 256) continue;
            const int FR = fh * fw, nb1 = (FR + 127) / 128, nb2 = (th * tw + 127) / 128;
            const int d1_cols = a.has_expand ? nb1 * 64 : 0;
            if (d1_cols + nb2 * n2 > 512) continue;
            const int stage = kin * 8192 * (a.has_expand ? 1 : 0) + n2 * 128;
            const size_t fixed = static_cast<size_t>(kin) * nb1 * kPlane + (a.has_expand ? nb1 * kPlane : 0) + static_cast<size_t>(nb2) * kPlane +
                                 4096 + static_cast<size_t>(chunks * 64 + n2) * 4 + 4096;
            // the output staging buffer (one 64-channel plane per 128-row block) if it fits beside two ring stages
            int out_planes = (a.Cout + 63) / 64;
            size_t so_bytes = static_cast<size_t>(out_planes) * nb2 * kPlane;
            if (fixed + so_bytes + 2 * static_cast<size_t>(stage) > static_cast<size_t>(kMaxSmem)) {
                out_planes = 0;
                so_bytes = 0;
            }
            int stages = 3;
            while (stages > 2 && fixed + so_bytes + static_cast<size_t>(stages) * stage > static_cast<size_t>(kMaxSmem)) stages--;
            if (fixed + so_bytes + static_cast<size_t>(stages) * stage > static_cast<size_t>(kMaxSmem)) continue;
            const int tiles_h = (Ho + th - 1) / th, tiles_w = (Wo + tw - 1) / tw;
            const long long n_tiles = static_cast<long long>(a.N) * tiles_h * tiles_w;
            if (n_tiles > 0x7fffffffLL) continue;
            const long long waves = (n_tiles + sm_count - 1) / sm_count;
            // per chunk: epilogue-1 rows + depthwise items on 256 threads, plus hand-off latency
            const double per_chunk = (a.has_expand ? nb1 * 128 * 1.5 : 0.0) + th * tw * 4.0 + 2500.0;
            // epilogue 2: staged tiles leave by TMA; direct stores touch one cache line per thread and instruction
            const double epi2 = th * tw * (n2 / 16.0) * (out_planes > 0 ? 1.0 : 4.0);
            const double cost = static_cast<double>(waves) * (chunks * per_chunk + epi2 + 3000.0);
            if (best_cost < 0 || cost < best_cost) {
                best_cost = cost;
                best.th = th; best.tw = tw; best.fh = fh; best.fw = fw; best.nb1 = nb1; best.nb2 = nb2;
                best.tiles_h = tiles_h; best.tiles_w = tiles_w; best.n_tiles = static_cast<int>(n_tiles);
                best.stages = stages; best.stage_bytes = stage;
                best.smem_bytes = fixed + so_bytes + static_cast<size_t>(stages) * stage;
                best.out_planes = out_planes;
                best.redundancy = static_cast<double>(FR) / (std::min(th, Ho) * a.stride * std::min(tw, Wo) * a.stride);
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
    MbParams p;
    std::memset(&p, 0, sizeof(p));
    p.N = a.N; p.H = a.H; p.W = a.W; p.Cin = a.Cin; p.hid = a.hid; p.Cout = a.Cout; p.stride = a.stride;
    p.Ho = (a.H + 2 - 3) / a.stride + 1; p.Wo = (a.W + 2 - 3) / a.stride + 1;
    p.has_expand = a.has_expand; p.act1 = a.act1; p.act2 = a.act2; p.act3 = a.act3;
    p.th = t.th; p.tw = t.tw; p.fh = t.fh; p.fw = t.fw; p.FR = t.fh * t.fw; p.nb1 = t.nb1; p.nb2 = t.nb2;
    p.tiles_h = t.tiles_h; p.tiles_w = t.tiles_w; p.n_tiles = t.n_tiles;
    p.kin = (a.Cin + 63) / 64; p.chunks = (a.hid + 63) / 64; p.n2_pad = pad16(a.Cout);
    p.ksteps_in_last = ((a.Cin - (p.kin - 1) * 64) + 15) / 16;
    p.x_off = 0;
    p.h_off = p.kin * p.nb1 * kPlane;
    p.hd_off = p.h_off + (a.has_expand ? p.nb1 * kPlane : 0);
    p.ring_off = p.hd_off + p.nb2 * kPlane;
    p.stage_bytes = t.stage_bytes; p.stages = t.stages;
    p.dw_off = p.ring_off + p.stages * p.stage_bytes;
    p.dw_off = (p.dw_off + 1023) / 1024 * 1024;
    p.bias_off = p.dw_off + 4096;
    p.so_planes = t.out_planes;
    p.so_off = (p.bias_off + (p.chunks * 64 + p.n2_pad) * 4 + 1023) / 1024 * 1024;
    p.d2_col = a.has_expand ? p.nb1 * 64 : 0;
    p.w2_off = a.has_expand ? p.kin * 8192 : 0;
    p.n_split = p.n2_pad > 256 ? 2 : 1;
    p.n_each = p.n2_pad / p.n_split;
    p.wd = static_cast<const __half*>(a.wd); p.b1 = a.b1; p.bd = a.bd; p.b2 = a.b2;
    p.res = static_cast<const __half*>(a.res); p.out = static_cast<__half*>(a.y); p.status = status_dev;
    {
        const uint64_t dims[4] = {static_cast<uint64_t>(a.Cin), static_cast<uint64_t>(a.W), static_cast<uint64_t>(a.H), static_cast<uint64_t>(a.N)};
        const uint64_t strides[3] = {static_cast<uint64_t>(a.Cin) * 2, static_cast<uint64_t>(a.W) * a.Cin * 2,
                                     static_cast<uint64_t>(a.H) * a.W * a.Cin * 2};
        const uint32_t box[4] = {64, static_cast<uint32_t>(t.fw), static_cast<uint32_t>(t.fh), 1};
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
    const size_t smem = std::max<size_t>(static_cast<size_t>(p.so_off) + static_cast<size_t>(p.so_planes) * p.nb2 * kPlane + 1024, 120 * 1024);
    if (smem > static_cast<size_t>(kMaxSmem)) return DLF_E_PLAN;
    cudaError_t e = launch_kernel(mbconv_tc_kernel, grid, kThreads, smem, s, p);
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

}  // namespace dlf
