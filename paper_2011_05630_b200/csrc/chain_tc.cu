// Fused fusion-group kernel: a chain of stride-1, size-keeping dense convolutions (3x3 pad 1 or
// 1x1) with bias / activation after each, optional residual and 2x2 max-pool on the last one,
// executed by ONE kernel whose intermediate feature maps never leave the SM (Sec. III-B of the
// paper: a fused layer's output is produced on chip and reused at once; Sec. IV-B: a spatial
// tile of a fused block recomputes its halo).
//
// Work item = (image, output tile th x tw of the last layer).  The tile's receptive-field frame
// (th + 2 halo) x (tw + 2 halo), halo = sum of the paddings, is loaded ONCE by TMA (zero fill
// outside the image = the first layer's padding) as a pixel-linear buffer: row q = fy*pitch + fx
// holds one pixel's 64 channels (128 bytes, 128-byte swizzle); wider layers use several planes.
// In that layout tap (r, s) of a 3x3 layer is the same buffer shifted by (r-1)*pitch + (s-1)
// rows, so every layer - the first included - feeds the tensor cores straight from the resident
// tile through a shifted shared-memory descriptor: no im2col, no per-tap reload.  A layer's M
// dimension is the linear range of frame positions it must produce (wrap-around columns are
// computed and ignored); its accumulators (up to 512 TMEM columns) are drained by four epilogue
// warps that add the bias, apply the activation, round to fp16, force positions outside the
// image to zero (they are the next layer's padding) and write the next layer's operand tile back
// to shared memory.  Weights stream through a TMA ring, once per layer per tile.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstring>

#include "internal.h"
#include "ptx.cuh"

namespace dlf {

namespace {

constexpr int kThreads = 192;
constexpr int kMaxSmem = 232448 - 1024;  // dynamic part: the 227 KB per-CTA limit minus the static barriers

struct ChainLayerP {
    int cin, cout, k, pad, act;
    int n_pad;      // cout rounded up to 16 (UMMA N)
    int slot;       // TMEM columns per 128-row block: n_pad rounded up to 32
    int kchunks;    // ceil(cin / 64)
    int ksteps_last;
    int cum_pad;    // sum of paddings up to and including this layer
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
    int buf_bytes;                  // planes_max * plane_bytes
    int in_planes;
    int stages, stage_bytes;
    int pool, base_offset_mode;
    int cout_last;
    const __half* res;
    __half* out;
    int* status;
};

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__global__ void __launch_bounds__(kThreads, 1) chain_tc_kernel(const __grid_constant__ ChainParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t wfull_bar[8], wempty_bar[8], in_full_bar, in_empty_bar, acc_full_bar, epi_done_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sbase = smem_raw + (base - smem_u32(smem_raw));
    // layout: [buf0][buf1][weight ring]
    const uint32_t ring_off = 2u * p.buf_bytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = &abort_s;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int i = 0; i < p.stages; i++) {
            mbar_init(&wfull_bar[i], 1);
            mbar_init(&wempty_bar[i], 1);
        }
        mbar_init(&in_full_bar, 1);
        mbar_init(&in_empty_bar, 1);
        mbar_init(&acc_full_bar, 1);
        mbar_init(&epi_done_bar, 4);
        fence_barrier_init();
        tma_prefetch_desc(&p.tmx);
    }
    if (warp == 1) {
        tmem_alloc(&tmem_base_s, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_s;
    const int frame_rows = p.rows * p.pitch;

    if (warp == 0) {
        // ---- producer ----------------------------------------------------------------------------------
        if (lane == 0) {
            uint32_t wit = 0, tile_i = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x, tile_i++) {
                const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h, n = t / (p.tiles_w * p.tiles_h);
                ok = mbar_wait(&in_empty_bar, (tile_i & 1u) ^ 1u, abort_flag, p.status, 0x100 | (blockIdx.x << 12));
                if (!ok) break;
                mbar_expect_tx(&in_full_bar, static_cast<uint32_t>(p.in_planes) * frame_rows * 128u);
                for (int pl = 0; pl < p.in_planes; pl++)
                    tma_load_4d(sbase + static_cast<size_t>(pl) * p.plane_bytes, &p.tmx, &in_full_bar, pl * 64,
                                txi * p.tw - p.halo, tyi * p.th - p.halo, n);
                for (int l = 0; l < p.n_layers && ok; l++) {
                    const ChainLayerP& L = p.L[l];
                    const int c = L.cum_pad;
                    const int range = (p.rows - 2 * c - 1) * p.pitch + (p.pitch - 2 * c);
                    const int nb = (range + 127) / 128, per_pass = 512 / L.slot;
                    const int passes = (nb + per_pass - 1) / per_pass;
                    const uint32_t bytes = static_cast<uint32_t>(L.n_pad) * 128u;
                    for (int ps = 0; ps < passes && ok; ps++)
                        for (int tap = 0; tap < L.k * L.k && ok; tap++)
                            for (int kc = 0; kc < L.kchunks; kc++, wit++) {
                                const int st = wit % p.stages;
                                ok = mbar_wait(&wempty_bar[st], ((wit / p.stages) & 1u) ^ 1u, abort_flag, p.status,
                                               0x200 | (blockIdx.x << 12));
                                if (!ok) break;
                                mbar_expect_tx(&wfull_bar[st], bytes);
                                tma_load_3d(sbase + ring_off + static_cast<size_t>(st) * p.stage_bytes, &p.tmw[l],
                                            &wfull_bar[st], kc * 64, tap, 0);
                            }
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer -----------------------------------------------------------------------------------
        if (lane == 0) {
            uint32_t wit = 0, tile_i = 0, pass_i = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x, tile_i++) {
                ok = mbar_wait(&in_full_bar, tile_i & 1u, abort_flag, p.status, 0x300 | (blockIdx.x << 12));
                if (!ok) break;
                for (int l = 0; l < p.n_layers && ok; l++) {
                    const ChainLayerP& L = p.L[l];
                    const int c = L.cum_pad;
                    const int qs = c * p.pitch + c;
                    const int range = (p.rows - 2 * c - 1) * p.pitch + (p.pitch - 2 * c);
                    const int nb = (range + 127) / 128, per_pass = 512 / L.slot;
                    const uint32_t idesc = umma_idesc_f16(L.n_pad);
                    const uint32_t abuf = base + (l & 1) * p.buf_bytes;
                    for (int b0 = 0; b0 < nb && ok; b0 += per_pass, pass_i++) {
                        const int nblk = min(per_pass, nb - b0);
                        if (pass_i > 0) {
                            // previous pass drained: TMEM is free and its shared-memory output is visible
                            ok = mbar_wait(&epi_done_bar, (pass_i - 1) & 1u, abort_flag, p.status, 0x400 | (blockIdx.x << 12));
                            if (!ok) break;
                        }
                        tc_fence_after_sync();
                        for (int tap = 0; tap < L.k * L.k && ok; tap++) {
                            const int r = tap / L.k, s = tap % L.k;
                            const int shift = (r - L.pad) * p.pitch + (s - L.pad);
                            for (int kc = 0; kc < L.kchunks; kc++, wit++) {
                                const int st = wit % p.stages;
                                ok = mbar_wait(&wfull_bar[st], (wit / p.stages) & 1u, abort_flag, p.status,
                                               0x500 | (blockIdx.x << 12));
                                if (!ok) break;
                                tc_fence_after_sync();
                                const uint32_t wsm = base + ring_off + st * p.stage_bytes;
                                const int ksteps = (kc == L.kchunks - 1) ? L.ksteps_last : 4;
                                for (int b = 0; b < nblk; b++) {
                                    const uint32_t arow = abuf + kc * p.plane_bytes + (qs + (b0 + b) * 128 + shift) * 128;
                                    const uint32_t bo = p.base_offset_mode ? ((arow >> 7) & 7u) : 0u;
                                    const uint32_t d_tmem = tmem_base + b * L.slot;
                                    for (int ks = 0; ks < ksteps; ks++)
                                        umma_f16(d_tmem, umma_desc_sw128(arow + ks * 32, bo),
                                                 umma_desc_sw128(wsm + ks * 32, 0), idesc, (tap | kc | ks) != 0);
                                }
                                umma_commit(&wempty_bar[st]);
                            }
                        }
                        if (ok) {
                            umma_commit(&acc_full_bar);
                            // an odd-length chain reads the input buffer last in its final layer
                            if (l == p.n_layers - 1 && b0 + per_pass >= nb && (p.n_layers & 1)) umma_commit(&in_empty_bar);
                        }
                    }
                }
            }
        }
    } else {
        // ---- epilogue warps (128 threads = 128 TMEM lanes) -------------------------------------------------
        const int q4 = warp & 3;
        const int row = q4 * 32 + lane;
        const int et = threadIdx.x - 64;  // 0..127
        uint32_t pass_i = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.n_tiles && ok; t += gridDim.x) {
            const int txi = t % p.tiles_w, tyi = (t / p.tiles_w) % p.tiles_h, n = t / (p.tiles_w * p.tiles_h);
            const int gy0 = tyi * p.th - p.halo, gx0 = txi * p.tw - p.halo;
            for (int l = 0; l < p.n_layers && ok; l++) {
                const ChainLayerP& L = p.L[l];
                const bool last = (l == p.n_layers - 1);
                const int c = L.cum_pad;
                const int qs = c * p.pitch + c;
                const int range = (p.rows - 2 * c - 1) * p.pitch + (p.pitch - 2 * c);
                const int nb = (range + 127) / 128, per_pass = 512 / L.slot;
                uint8_t* obuf = sbase + ((l + 1) & 1) * p.buf_bytes;
                for (int b0 = 0; b0 < nb && ok; b0 += per_pass, pass_i++) {
                    const int nblk = min(per_pass, nb - b0);
                    ok = mbar_wait(&acc_full_bar, pass_i & 1u, abort_flag, p.status, 0x600 | (blockIdx.x << 12));
                    if (!ok) break;
                    tc_fence_after_sync();
                    for (int b = 0; b < nblk; b++) {
                        const int q = qs + (b0 + b) * 128 + row;
                        const int fy = q / p.pitch, fx = q - fy * p.pitch;
                        const int gy = gy0 + fy, gx = gx0 + fx;
                        const bool in_range = q < qs + range;
                        const bool in_img = gy >= 0 && gy < p.H && gx >= 0 && gx < p.W;
                        const long long gpix = (static_cast<long long>(n) * p.H + gy) * p.W + gx;
                        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q4 * 32) << 16) + b * L.slot;
                        for (int cc = 0; cc < L.n_pad; cc += 16) {
                            float v[16];
                            __syncwarp();  // the aligned TMEM load needs the whole warp converged
                            tmem_ld16(taddr + cc, v);
                            if (!in_range) continue;
                            uint32_t packed[8];
#pragma unroll
                            for (int e = 0; e < 8; e++) {
                                const int co = cc + 2 * e;
                                float a0 = 0.0f, a1 = 0.0f;
                                if (in_img && co < L.cout) {  // cout is a multiple of 8: pairs never straddle
                                    a0 = v[2 * e] + __ldg(L.bias + co);
                                    a1 = v[2 * e + 1] + __ldg(L.bias + co + 1);
                                    if (last && p.res != nullptr) {
                                        const __half2 rh = __ldg(reinterpret_cast<const __half2*>(p.res + gpix * L.cout + co));
                                        const float2 rf = __half22float2(rh);
                                        a0 += rf.x;
                                        a1 += rf.y;
                                    }
                                    a0 = apply_act(a0, L.act);
                                    a1 = apply_act(a1, L.act);
                                }
                                packed[e] = pack_half2(a0, a1);
                            }
#pragma unroll
                            for (int h8 = 0; h8 < 2; h8++) {
                                const int g8 = (cc >> 3) + h8;  // 8-channel group index
                                uint8_t* dst = obuf + static_cast<size_t>(g8 >> 3) * p.plane_bytes + static_cast<size_t>(q) * 128 +
                                               (((g8 & 7) ^ (q & 7)) << 4);
                                *reinterpret_cast<uint4*>(dst) =
                                    make_uint4(packed[h8 * 4], packed[h8 * 4 + 1], packed[h8 * 4 + 2], packed[h8 * 4 + 3]);
                            }
                        }
                    }
                    fence_proxy_async_smem();  // the next layer's UMMAs read these rows through the async proxy
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&epi_done_bar);
                }
            }
            if (!ok) break;
            // ---- copy the tile out (coalesced 16-byte stores), pooling 2x2 if asked ----------------
            epi_bar_sync();
            {
                const uint8_t* obuf = sbase + (p.n_layers & 1) * p.buf_bytes;
                const int c8n = p.cout_last / 8;
                const int win = p.pool ? 2 : 1;
                const int oth = p.th / win, otw = p.tw / win;
                const int Ho = p.H / win, Wo = p.W / win;
                const int total = oth * otw * c8n;
                for (int i = et; i < total; i += 128) {
                    const int g8 = i % c8n;
                    const int ox = (i / c8n) % otw, oy = i / (c8n * otw);
                    const int gy = tyi * oth + oy, gx = txi * otw + ox;
                    if (gy >= Ho || gx >= Wo) continue;
                    uint4 best = make_uint4(0, 0, 0, 0);
                    for (int wy = 0; wy < win; wy++)
                        for (int wx = 0; wx < win; wx++) {
                            const int q = (p.halo + oy * win + wy) * p.pitch + p.halo + ox * win + wx;
                            const uint4 vv = *reinterpret_cast<const uint4*>(obuf + static_cast<size_t>(g8 >> 3) * p.plane_bytes +
                                                                             static_cast<size_t>(q) * 128 + (((g8 & 7) ^ (q & 7)) << 4));
                            if (wy == 0 && wx == 0) {
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
            }
            epi_bar_sync();
            // an even-length chain overwrites the input buffer in its last epilogue
            if (!(p.n_layers & 1) && et == 0) mbar_arrive(&in_empty_bar);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        if (abort_s) __nanosleep(20000);
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

int planes_of(int c) { return (c + 63) / 64; }

// Rows one activation plane must hold: the frame itself, plus what the last 128-row block of a
// layer may touch past it (its own rows when written, its farthest tap when read).
int rows_alloc_of(const ChainArgs& a, int rows, int pitch) {
    int need = rows * pitch, c = 0;
    for (int l = 0; l < a.n_layers; l++) {
        const int pad = a.k[l] / 2;
        c += pad;
        const int qs = c * pitch + c;
        const int range = (rows - 2 * c - 1) * pitch + (pitch - 2 * c);
        const int nb = (range + 127) / 128;
        need = std::max(need, qs + nb * 128 + pad * pitch + pad);
    }
    return (need + 7) / 8 * 8;
}

}  // namespace

// Picks the output tile from the SM count: among the tile shapes whose buffers fit in shared
// memory, the one with the least estimated time = waves x (tensor-core work of one tile,
// counted in 128-row blocks, plus a fixed per-tile cost).
ChainTiling chain_tc_tiling(const ChainArgs& a, int sm_count, int device_sms) {
    ChainTiling best{};
    best.ok = false;
    (void)device_sms;
    if (a.n_layers < 1 || a.n_layers > kMaxChain) return best;
    int halo = 0, planes_max = 0, nmax = 0;
    for (int l = 0; l < a.n_layers; l++) {
        if (a.k[l] != 1 && a.k[l] != 3) return best;
        if (a.cin[l] % 8 || a.cout[l] % 8 || a.cout[l] > 256) return best;
        if (l > 0 && a.cin[l] != a.cout[l - 1]) return best;
        halo += a.k[l] / 2;
        planes_max = std::max(planes_max, std::max(planes_of(a.cin[l]), planes_of((a.cout[l] + 15) / 16 * 16)));
        nmax = std::max(nmax, (a.cout[l] + 15) / 16 * 16);
    }
    const int stage_bytes = nmax * 128;
    static const int cand[] = {2, 4, 6, 8, 12, 16, 24, 32, 48, 64};
    double best_cost = -1.0;
    for (int th : cand)
        for (int tw : cand) {
            if (a.pool && ((th | tw) & 1)) continue;
            if (th > std::max(a.H, 2) * 2 || tw > std::max(a.W, 2) * 2) continue;
            const int rows = th + 2 * halo, pitch = tw + 2 * halo;
            if (rows > 256 || pitch > 256) continue;
            const int rows_alloc = rows_alloc_of(a, rows, pitch);
            const size_t buf = static_cast<size_t>(planes_max) * rows_alloc * 128;
            int stages = 8;
            while (stages > 2 && 2 * buf + static_cast<size_t>(stages) * stage_bytes + 1024 > kMaxSmem) stages--;
            if (2 * buf + static_cast<size_t>(stages) * stage_bytes + 1024 > kMaxSmem) continue;
            const int tiles_h = (a.H + th - 1) / th, tiles_w = (a.W + tw - 1) / tw;
            const long long n_tiles = static_cast<long long>(a.N) * tiles_h * tiles_w;
            if (n_tiles > 0x7fffffffLL) continue;
            const long long waves = (n_tiles + sm_count - 1) / sm_count;
            double work = 0.0, useful = 0.0, computed = 0.0;
            int c = 0;
            for (int l = 0; l < a.n_layers; l++) {
                c += a.k[l] / 2;
                const int range = (rows - 2 * c - 1) * pitch + (pitch - 2 * c);
                const int nb = (range + 127) / 128;
                const double kk = static_cast<double>(a.k[l]) * a.k[l] * ((a.cin[l] + 15) / 16 * 16);
                const int npad = (a.cout[l] + 15) / 16 * 16;
                const int slot = (npad + 31) / 32 * 32;
                const int passes = (nb + 512 / slot - 1) / (512 / slot);
                work += nb * 128.0 * kk * npad + passes * 2.0e5;
                computed += nb * 128.0 * kk * npad;
                useful += static_cast<double>(std::min(th, a.H)) * std::min(tw, a.W) * a.k[l] * a.k[l] * a.cin[l] * a.cout[l];
            }
            work += static_cast<double>(rows) * pitch * planes_max * 64 * 40.0 + 4.0e5;  // input load + fixed cost
            const double cost = static_cast<double>(waves) * work;
            if (best_cost < 0 || cost < best_cost) {
                best_cost = cost;
                best.th = th; best.tw = tw; best.halo = halo; best.pitch = pitch; best.rows = rows;
                best.tiles_h = tiles_h; best.tiles_w = tiles_w; best.n_tiles = static_cast<int>(n_tiles);
                best.stages = stages;
                best.smem_bytes = 2 * buf + static_cast<size_t>(stages) * stage_bytes + 1024;
                best.tmem_cols = 512;
                best.redundancy = computed / useful;
                best.ok = true;
            }
        }
    return best;
}

int launch_chain_tc(const ChainArgs& a, const ChainTiling& t, int sm_count, int base_offset_mode, int* status_dev,
                    cudaStream_t s) {
    if (!t.ok) return DLF_E_PLAN;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(chain_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e != cudaSuccess) return cuda_fail(e);
        attr_set = true;
    }
    ChainParams p;
    std::memset(&p, 0, sizeof(p));
    p.n_layers = a.n_layers;
    p.N = a.N; p.H = a.H; p.W = a.W;
    p.th = t.th; p.tw = t.tw; p.halo = t.halo; p.pitch = t.pitch; p.rows = t.rows;
    p.tiles_h = t.tiles_h; p.tiles_w = t.tiles_w; p.n_tiles = t.n_tiles;
    int planes_max = 0, nmax = 0, cum = 0;
    for (int l = 0; l < a.n_layers; l++) {
        ChainLayerP& L = p.L[l];
        L.cin = a.cin[l]; L.cout = a.cout[l]; L.k = a.k[l]; L.pad = a.k[l] / 2; L.act = a.act[l];
        L.n_pad = (a.cout[l] + 15) / 16 * 16;
        L.slot = (L.n_pad + 31) / 32 * 32;
        L.kchunks = planes_of(a.cin[l]);
        L.ksteps_last = ((a.cin[l] - (L.kchunks - 1) * 64) + 15) / 16;
        cum += L.pad;
        L.cum_pad = cum;
        L.bias = a.bias[l];
        planes_max = std::max(planes_max, std::max(planes_of(a.cin[l]), planes_of(L.n_pad)));
        nmax = std::max(nmax, L.n_pad);
        const uint64_t taps = static_cast<uint64_t>(a.k[l]) * a.k[l];
        const uint64_t dims[3] = {static_cast<uint64_t>(a.cin[l]), taps, static_cast<uint64_t>(a.cout[l])};
        const uint64_t strides[2] = {static_cast<uint64_t>(a.cin[l]) * 2, taps * a.cin[l] * 2};
        const uint32_t box[3] = {64, 1, static_cast<uint32_t>(L.n_pad)};
        const uint32_t es[3] = {1, 1, 1};
        int rc = encode_tmap(&p.tmw[l], a.w[l], 3, dims, strides, box, es);
        if (rc) return rc;
    }
    const int rows_alloc = rows_alloc_of(a, t.rows, t.pitch);
    p.plane_bytes = rows_alloc * 128;
    p.buf_bytes = planes_max * p.plane_bytes;
    p.in_planes = planes_of(a.cin[0]);
    p.stages = t.stages;
    p.stage_bytes = nmax * 128;
    p.pool = a.pool;
    p.base_offset_mode = base_offset_mode;
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
    chain_tc_kernel<<<grid, kThreads, smem, s>>>(p);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

}  // namespace dlf
