// Single-layer implicit-GEMM convolution on the tcgen05 tensor cores (the kernel of the
// no-fusion plan, and of every group that holds one dense convolution).
//
//   D[m, n] = sum over (tap, ci) of A_tap[m, ci] * W[n, tap, ci]        (Eq. 1 counts these MACs)
//   M = 128 output pixels (a TN x TH x TW patch), N = up to 256 output channels, K = taps x C_in.
//
// A persistent grid of `sm_count` CTAs (the SM-count knob) walks the (pixel tile, channel tile)
// work list.  Per CTA: one producer thread issues TMA tiled loads (the tap's shifted, strided
// window of the NHWC input, zero-filled outside the image = the convolution's padding; and the
// tap's [C_out][64] weight slab) into a ring of 128-byte-swizzled stages; one thread issues
// tcgen05.mma (fp16 x fp16 -> fp32) into one of two TMEM accumulators; four epilogue warps read
// the other accumulator with tcgen05.ld and apply bias, residual, activation, the fp16 rounding
// and the optional 2x2 max-pool (warp shuffles) before 16-byte global stores.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>

#include "internal.h"
#include "ptx.cuh"

namespace dlf {

namespace {

constexpr int kThreads = 192;
constexpr int kABytes = 128 * 128;  // 128 pixels x 64 fp16
constexpr int kMaxSmem = 232448 - 1024;  // dynamic part: the 227 KB per-CTA limit minus the static barriers

struct ConvTcParams {
    int N, Ho, Wo, Cout;
    int kh, kw, stride, pad;
    int TW, TH, TN, tiles_w, tiles_h, tiles_n;
    int BN, n_tiles_n, acc_stride;
    int kchunks, ksteps_last;
    int act, pool, stages;
    int n_work;
    uint32_t tmem_cols;
    const float* bias;
    const __half* res;
    __half* out;
    int* status;
};

struct TileCoord {
    int n0, ho0, wo0, co0;
};

__device__ __forceinline__ TileCoord decode_work(const ConvTcParams& p, int t) {
    TileCoord c;
    const int nt = t % p.n_tiles_n;
    int mt = t / p.n_tiles_n;
    c.co0 = nt * p.BN;
    c.wo0 = (mt % p.tiles_w) * p.TW;
    mt /= p.tiles_w;
    c.ho0 = (mt % p.tiles_h) * p.TH;
    c.n0 = (mt / p.tiles_h) * p.TN;
    return c;
}

__global__ void __launch_bounds__(kThreads, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tmw, const ConvTcParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[8], empty_bar[8], tfull_bar[2], tempty_bar[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    if (threadIdx.x == 0) DLF_TRACE_POINT(p.status, 0);
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* stage0 = smem_raw + (base - smem_u32(smem_raw));
    const int stage_bytes = kABytes + p.BN * 128;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = &abort_s;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int i = 0; i < p.stages; i++) {
            mbar_init(&full_bar[i], 1);
            mbar_init(&empty_bar[i], 1);
        }
        for (int i = 0; i < 2; i++) {
            mbar_init(&tfull_bar[i], 1);
            mbar_init(&tempty_bar[i], 4);
        }
        fence_barrier_init();
        tma_prefetch_desc(&tmx);
        tma_prefetch_desc(&tmw);
    }
    if (warp == 1) {
        tmem_alloc(&tmem_base_s, p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (threadIdx.x == 0) DLF_TRACE_POINT(p.status, 1);
    const uint32_t tmem_base = tmem_base_s;
    const int taps = p.kh * p.kw;
    const int k_iters = taps * p.kchunks;

    if (warp == 0) {
        // ---- producer: TMA loads into the stage ring ------------------------------------------
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.n_work && ok; t += gridDim.x) {
                const TileCoord c = decode_work(p, t);
                for (int tap = 0; tap < taps && ok; tap++) {
                    const int r = tap / p.kw, s = tap % p.kw;
                    for (int kc = 0; kc < p.kchunks; kc++, it++) {
                        const int st = it % p.stages;
                        ok = mbar_wait(&empty_bar[st], ((it / p.stages) & 1u) ^ 1u, abort_flag, p.status,
                                       0x100 | (blockIdx.x << 12));
                        if (!ok) break;
                        uint8_t* sa = stage0 + static_cast<size_t>(st) * stage_bytes;
                        mbar_expect_tx(&full_bar[st], static_cast<uint32_t>(stage_bytes));
                        tma_load_4d(sa, &tmx, &full_bar[st], kc * 64, c.wo0 * p.stride - p.pad + s,
                                    c.ho0 * p.stride - p.pad + r, c.n0);
                        tma_load_3d(sa + kABytes, &tmw, &full_bar[st], kc * 64, tap, c.co0);
                        if (it == 0) DLF_TRACE_POINT(p.status, 2);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer ---------------------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f16(p.BN);
            uint32_t it = 0, j = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.n_work && ok; t += gridDim.x, j++) {
                const uint32_t acc = j & 1u;
                ok = mbar_wait(&tempty_bar[acc], ((j >> 1) & 1u) ^ 1u, abort_flag, p.status, 0x200 | (blockIdx.x << 12));
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * p.acc_stride;
                for (int ki = 0; ki < k_iters; ki++, it++) {
                    const int st = it % p.stages;
                    ok = mbar_wait(&full_bar[st], (it / p.stages) & 1u, abort_flag, p.status, 0x300 | (blockIdx.x << 12));
                    if (!ok) break;
                    if (it == 0) DLF_TRACE_POINT(p.status, 3);
                    tc_fence_after_sync();
                    const uint32_t sa = base + st * stage_bytes;
                    const int ksteps = ((ki % p.kchunks) == p.kchunks - 1) ? p.ksteps_last : 4;
                    for (int ks = 0; ks < ksteps; ks++) {
                        umma_f16(d_tmem, umma_desc_sw128(sa + ks * 32, 0), umma_desc_sw128(sa + kABytes + ks * 32, 0),
                                 idesc, (ki | ks) != 0);
                    }
                    umma_commit(&empty_bar[st]);  // frees the stage once these MMAs have read it
                }
                if (ok) umma_commit(&tfull_bar[acc]);
                if (j == 0) DLF_TRACE_POINT(p.status, 4);
            }
        }
    } else {
        // ---- epilogue warps ---------------------------------------------------------------------------
        const int q = warp & 3;  // TMEM lane quarter this warp may read
        const int m = q * 32 + lane;
        const int tw = m % p.TW, th = (m / p.TW) % p.TH, tn = m / (p.TW * p.TH);
        const int Hp = p.pool ? p.Ho / 2 : p.Ho, Wp = p.pool ? p.Wo / 2 : p.Wo;
        uint32_t j = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.n_work && ok; t += gridDim.x, j++) {
            const TileCoord c = decode_work(p, t);
            const uint32_t acc = j & 1u;
            ok = mbar_wait(&tfull_bar[acc], (j >> 1) & 1u, abort_flag, p.status, 0x400 | (blockIdx.x << 12));
            if (!ok) break;
            if (j == 0 && threadIdx.x == 64) DLF_TRACE_POINT(p.status, 5);
            tc_fence_after_sync();
            const int n = c.n0 + tn, ho = c.ho0 + th, wo = c.wo0 + tw;
            const bool valid = n < p.N && ho < p.Ho && wo < p.Wo;
            const long long pix = (static_cast<long long>(n) * p.Ho + ho) * p.Wo + wo;
            const long long opix = p.pool ? (static_cast<long long>(n) * Hp + (ho >> 1)) * Wp + (wo >> 1) : pix;
            const bool writer = valid && (!p.pool || (((ho | wo) & 1) == 0 && (ho >> 1) < Hp && (wo >> 1) < Wp));
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * p.acc_stride;
            const int ncols = min(p.BN, p.Cout - c.co0);
            for (int cc = 0; cc < ncols; cc += 16) {
                float v[16];
                __syncwarp();  // the aligned TMEM load needs the whole warp converged
                tmem_ld16(taddr + cc, v);
                const int co = c.co0 + cc;
                const int nv = min(16, p.Cout - co);  // 8 or 16
#pragma unroll
                for (int h8 = 0; h8 < 2; h8++) {
                    if (h8 * 8 >= nv) break;
                    const float4 b0 = __ldg(reinterpret_cast<const float4*>(p.bias + co + h8 * 8));
                    const float4 b1 = __ldg(reinterpret_cast<const float4*>(p.bias + co + h8 * 8 + 4));
                    float* vv = v + h8 * 8;
                    vv[0] += b0.x; vv[1] += b0.y; vv[2] += b0.z; vv[3] += b0.w;
                    vv[4] += b1.x; vv[5] += b1.y; vv[6] += b1.z; vv[7] += b1.w;
                    if (p.res != nullptr && valid) {
                        const uint4 rv = __ldg(reinterpret_cast<const uint4*>(p.res + pix * p.Cout + co + h8 * 8));
                        const __half2* rh = reinterpret_cast<const __half2*>(&rv);
#pragma unroll
                        for (int e = 0; e < 4; e++) {
                            const float2 f = __half22float2(rh[e]);
                            vv[2 * e] += f.x;
                            vv[2 * e + 1] += f.y;
                        }
                    }
                    uint4 o;
                    uint32_t* ou = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                    for (int e = 0; e < 4; e++) {
                        float a0 = apply_act(vv[2 * e], p.act), a1 = apply_act(vv[2 * e + 1], p.act);
                        if (p.pool) {
                            // round first, then take the max over the 2x2 window held by this warp
                            __half2 hv = __floats2half2_rn(a0, a1);
                            __half2 o1 = __shfl_xor_sync(0xffffffffu, hv, 1);
                            hv = __hmax2(hv, o1);
                            o1 = __shfl_xor_sync(0xffffffffu, hv, p.TW);
                            hv = __hmax2(hv, o1);
                            ou[e] = *reinterpret_cast<uint32_t*>(&hv);
                        } else {
                            ou[e] = pack_half2(a0, a1);
                        }
                    }
                    if (writer) *reinterpret_cast<uint4*>(p.out + opix * p.Cout + co + h8 * 8) = o;
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tempty_bar[acc]);
            if (j == 0 && threadIdx.x == 64) DLF_TRACE_POINT(p.status, 6);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        if (abort_s) __nanosleep(20000);  // let copies in flight land before the CTA retires
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, p.tmem_cols);
        if (lane == 0) DLF_TRACE_POINT(p.status, 7);
    }
}

struct Tile {
    int tw, th, tn;
};

Tile pick_tile(int N, int Ho, int Wo, int pool) {
    Tile best{16, 8, 1};
    long long best_tiles = -1;
    for (int tw = 128; tw >= 2; tw >>= 1) {
        if (pool && tw > 16) continue;
        for (int th = 128 / tw; th >= 1; th >>= 1) {
            if (pool && th < 2) continue;
            const int tn = 128 / (tw * th);
            const long long tiles = static_cast<long long>((Wo + tw - 1) / tw) * ((Ho + th - 1) / th) * ((N + tn - 1) / tn);
            if (best_tiles < 0 || tiles < best_tiles) {
                best_tiles = tiles;
                best = Tile{tw, th, tn};
            }
        }
    }
    return best;
}

}  // namespace

bool conv_tc_supported(const ConvArgs& a) {
    if (a.groups != 1) return false;
    if (a.Cin % 8 || a.Cout % 8) return false;
    if (a.stride < 1 || a.stride > 2) return false;
    if (a.kh * a.kw > 49) return false;
    if (a.N < 1 || a.Ho < 1 || a.Wo < 1) return false;
    return true;
}

int launch_conv_tc(const ConvArgs& a, int sm_count, int* status_dev, cudaStream_t s) {
    if (!conv_tc_supported(a)) return DLF_E_UNSUPPORTED;
    {
        int rc = conv_tc_init();
        if (rc) return rc;
    }
    ConvTcParams p{};
    p.N = a.N; p.Ho = a.Ho; p.Wo = a.Wo; p.Cout = a.Cout;
    p.kh = a.kh; p.kw = a.kw; p.stride = a.stride; p.pad = a.pad;
    const Tile tl = pick_tile(a.N, a.Ho, a.Wo, a.pool);
    p.TW = tl.tw; p.TH = tl.th; p.TN = tl.tn;
    p.tiles_w = (a.Wo + tl.tw - 1) / tl.tw;
    p.tiles_h = (a.Ho + tl.th - 1) / tl.th;
    p.tiles_n = (a.N + tl.tn - 1) / tl.tn;
    const int cout16 = (a.Cout + 15) / 16 * 16;
    p.n_tiles_n = (cout16 + 255) / 256;
    p.BN = ((cout16 + p.n_tiles_n - 1) / p.n_tiles_n + 15) / 16 * 16;
    p.kchunks = (a.Cin + 63) / 64;
    p.ksteps_last = ((a.Cin - (p.kchunks - 1) * 64) + 15) / 16;
    p.act = a.act; p.pool = a.pool;
    const int stage_bytes = kABytes + p.BN * 128;
    p.stages = std::min(6, (kMaxSmem - 1024) / stage_bytes);
    p.stages = std::max(1, std::min(p.stages, a.kh * a.kw * p.kchunks));
    const long long n_work = static_cast<long long>(p.tiles_w) * p.tiles_h * p.tiles_n * p.n_tiles_n;
    if (n_work > 0x7fffffffLL) return DLF_E_UNSUPPORTED;
    p.n_work = static_cast<int>(n_work);
    uint32_t cols = 32;
    p.acc_stride = (p.BN + 31) / 32 * 32;
    while (cols < static_cast<uint32_t>(2 * p.acc_stride)) cols <<= 1;
    p.tmem_cols = cols;
    p.bias = a.bias; p.res = static_cast<const __half*>(a.res); p.out = static_cast<__half*>(a.y);
    p.status = status_dev;

    CUtensorMap tmx, tmw;
    {
        const uint64_t dims[4] = {static_cast<uint64_t>(a.Cin), static_cast<uint64_t>(a.W), static_cast<uint64_t>(a.H),
                                  static_cast<uint64_t>(a.N)};
        const uint64_t strides[3] = {static_cast<uint64_t>(a.Cin) * 2, static_cast<uint64_t>(a.W) * a.Cin * 2,
                                     static_cast<uint64_t>(a.H) * a.W * a.Cin * 2};
        const uint32_t box[4] = {64, static_cast<uint32_t>(tl.tw * a.stride), static_cast<uint32_t>(tl.th * a.stride),
                                 static_cast<uint32_t>(tl.tn)};
        const uint32_t es[4] = {1, static_cast<uint32_t>(a.stride), static_cast<uint32_t>(a.stride), 1};
        int rc = encode_tmap(&tmx, a.x, 4, dims, strides, box, es);
        if (rc) return rc;
    }
    {
        const uint64_t taps = static_cast<uint64_t>(a.kh) * a.kw;
        const uint64_t dims[3] = {static_cast<uint64_t>(a.Cin), taps, static_cast<uint64_t>(a.Cout)};
        const uint64_t strides[2] = {static_cast<uint64_t>(a.Cin) * 2, taps * a.Cin * 2};
        const uint32_t box[3] = {64, 1, static_cast<uint32_t>(p.BN)};
        const uint32_t es[3] = {1, 1, 1};
        int rc = encode_tmap(&tmw, a.w, 3, dims, strides, box, es);
        if (rc) return rc;
    }
    const int grid = std::max(1, std::min(sm_count, p.n_work));
    const size_t smem = std::max<size_t>(static_cast<size_t>(p.stages) * stage_bytes + 1024, 120 * 1024);
    conv_tc_kernel<<<grid, kThreads, smem, s>>>(tmx, tmw, p);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

int conv_tc_init() {
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e != cudaSuccess) return cuda_fail(e);
        attr_set = true;
    }
    return DLF_OK;
}

}  // namespace dlf
