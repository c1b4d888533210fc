// First-layer ("stem") convolution on the tensor cores: C_in <= 4 (the RGB input), kernel up to
// 7x7, stride 1 or 2, up to 64 output channels, bias + activation.
//
// With three input channels a tap is only 6 bytes wide, far below what TMA can address (16-byte
// strides) or a UMMA K step can use, so the implicit-GEMM operand is built in shared memory by the
// CTA's own threads: for output pixel m and kernel row r the kw * C_in input values are contiguous
// in NHWC memory; they are gathered (zero outside the image) into K positions r*KR .. r*KR+kw*C_in-1
// of row m of a 128-byte-swizzled A tile (KR = kw*C_in rounded up to 8, K = kh*KR rounded up to 64).
// The weights are laid out the same way once per CTA.  One thread then issues the UMMAs
// (M = 128 pixels, N = C_out, K) into one of two TMEM accumulators while the same eight warps
// build the next tile and drain the previous one (bias, activation, fp16 rounding, staging tile,
// TMA store).  Eq. 1 counts kh*kw*C_in*C_out MACs per output pixel; the padded K positions hold
// zeros on both operands.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>

#include "internal.h"
#include "ptx.cuh"

namespace dlf {

namespace {

constexpr int kWorkWarps = 8;                 // warps 0..7 build A tiles and run the epilogue
constexpr int kMmaWarp = kWorkWarps;          // warp 8 issues the UMMAs and owns the TMEM allocation
constexpr int kThreads = 32 * (kWorkWarps + 1);
constexpr int kPlane = 128 * 128;             // one 64-wide K chunk of the A tile
constexpr int kMaxKChunks = 4;

struct StemParams {
    const __half* x;
    const __half* w;
    const float* bias;
    int* status;
    int N, H, W, Cin, Ho, Wo, Cout;
    int kh, kw, stride, pad, act;
    int KR, kchunks, BN;
    int TW, TH, TN, tiles_w, tiles_h, tiles_n, n_work;
};

__device__ __forceinline__ void work_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(32 * kWorkWarps) : "memory"); }

// CIN > 0: the channel count is a compile-time constant (the tap / channel index arithmetic of the
// gather folds away); CIN == 0: any channel count up to 4.
template <int CIN>
__global__ void __launch_bounds__(kThreads, 1) stem_tc_kernel(const __grid_constant__ CUtensorMap tmy, const StemParams p) {
    const int cin = CIN > 0 ? CIN : p.Cin;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t a_full_bar[2], t_full_bar[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ float bias_s[64];

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sbase = smem_raw + (base - smem_u32(smem_raw));
    // layout: A[2][kchunks][128 x 128 B] | B[kchunks][64 x 128 B] | staging [128 x 128 B]
    const int a_bytes = p.kchunks * kPlane;
    uint8_t* bsm = sbase + 2 * a_bytes;
    uint8_t* stage_out = bsm + p.kchunks * 8192;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = &abort_s;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int i = 0; i < 2; i++) {
            mbar_init(&a_full_bar[i], kWorkWarps);
            mbar_init(&t_full_bar[i], 1);
        }
        fence_barrier_init();
        tma_prefetch_desc(&tmy);
    }
    if (warp == kMmaWarp) {
        tmem_alloc(&tmem_base_s, 128);
        tmem_relinquish();
    }
    if (threadIdx.x < 64) bias_s[threadIdx.x] = threadIdx.x < p.Cout ? __ldg(p.bias + threadIdx.x) : 0.0f;
    // zero both A buffers (their K padding is never written again) and lay out the weights
    for (int i = threadIdx.x; i < (2 * a_bytes + p.kchunks * 8192) / 16; i += kThreads)
        reinterpret_cast<uint4*>(sbase)[i] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    {
        const int per_co = p.kh * p.kw * cin;
        for (int i = threadIdx.x; i < p.Cout * per_co; i += kThreads) {
            const int co = i / per_co, rem = i - co * per_co;
            const int r = rem / (p.kw * cin), sc = rem - r * (p.kw * cin);
            const int k = r * p.KR + sc;
            *reinterpret_cast<__half*>(bsm + (k >> 6) * 8192 + co * 128 + ((((k & 63) >> 3) ^ (co & 7)) << 4) + (k & 7) * 2) = p.w[i];
        }
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();
    pdl_wait();  // weights are constants; the input may come from the previous kernel
    const uint32_t tmem_base = tmem_base_s;

    if (warp == kMmaWarp) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f16(p.BN);
            uint32_t j = 0;
            for (int t = blockIdx.x; t < p.n_work; t += gridDim.x, j++) {
                const uint32_t b = j & 1u;
                if (!mbar_wait(&a_full_bar[b], (j >> 1) & 1u, abort_flag, p.status, 0x900 | (blockIdx.x << 12))) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + b * 64u;
                for (int kc = 0; kc < p.kchunks; kc++) {
                    const uint32_t a_lo = umma_desc_lo(base + b * a_bytes + kc * kPlane);
                    const uint32_t b_lo = umma_desc_lo(base + 2 * a_bytes + kc * 8192);
#pragma unroll
                    for (int ks = 0; ks < 4; ks++)
                        umma_f16_lo(d_tmem, a_lo + 2 * ks, kDescHiSw128, b_lo + 2 * ks, idesc, (kc | ks) != 0);
                }
                umma_commit(&t_full_bar[b]);
            }
        }
    } else {
        const int kwc = p.kw * cin;
        const int chunks_per_row = p.KR >> 3;
        const int q = warp & 3, half = warp >> 2;
        uint32_t j = 0;
        bool ok = true;
        int prev_t = -1;
        // software pipeline: build tile j, then drain tile j-1 while the tensor core works on tile j
        for (int t = blockIdx.x;; t += gridDim.x, j++) {
            const bool have = t < p.n_work;
            if (have) {
                int mt = t;
                const int wo0 = (mt % p.tiles_w) * p.TW;
                mt /= p.tiles_w;
                const int ho0 = (mt % p.tiles_h) * p.TH, n0 = (mt / p.tiles_h) * p.TN;
                uint8_t* abuf = sbase + (j & 1u) * a_bytes;
                for (int item = threadIdx.x; item < 128 * p.kh; item += 32 * kWorkWarps) {
                    const int m = item % 128, r = item / 128;
                    const int n = n0 + m / (p.TW * p.TH), ho = ho0 + (m / p.TW) % p.TH, wo = wo0 + m % p.TW;
                    const int hi = ho * p.stride - p.pad + r;
                    const bool row_ok = n < p.N && ho < p.Ho && wo < p.Wo && hi >= 0 && hi < p.H;
                    const int wi0 = wo * p.stride - p.pad;
                    const __half* src = p.x + ((static_cast<long long>(n) * p.H + hi) * p.W + wi0) * cin;
                    for (int ck = 0; ck < chunks_per_row; ck++) {
                        __align__(16) __half vals[8];
#pragma unroll
                        for (int e = 0; e < 8; e++) {
                            const int idx = ck * 8 + e;               // position inside this kernel row's K slice
                            const int wi = wi0 + idx / cin;
                            const bool in = row_ok && idx < kwc && wi >= 0 && wi < p.W;
                            vals[e] = in ? src[idx] : __ushort_as_half(0);
                        }
                        const int kchunk = r * chunks_per_row + ck;  // 16-byte chunk index along K
                        *reinterpret_cast<uint4*>(abuf + (kchunk >> 3) * kPlane + m * 128 + (((kchunk & 7) ^ (m & 7)) << 4)) =
                            *reinterpret_cast<const uint4*>(vals);
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&a_full_bar[j & 1u]);
            }
            if (prev_t >= 0) {
                const uint32_t jb = j - 1, b = jb & 1u;
                ok = mbar_wait(&t_full_bar[b], (jb >> 1) & 1u, abort_flag, p.status, 0xA00 | (blockIdx.x << 12));
                if (!ok) break;
                tc_fence_after_sync();
                int mt = prev_t;
                const int wo0 = (mt % p.tiles_w) * p.TW;
                mt /= p.tiles_w;
                const int ho0 = (mt % p.tiles_h) * p.TH, n0 = (mt / p.tiles_h) * p.TN;
                const int m = q * 32 + lane;
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + b * 64u;
                for (int cc = half * 32; cc < p.BN; cc += 64) {
                    float v[32];
                    __syncwarp();
                    const int nc = min(32, p.BN - cc);
                    if (nc == 32) tmem_ld32(taddr + cc, v);
                    else tmem_ld16(taddr + cc, v);
#pragma unroll
                    for (int g = 0; g < 4; g++) {
                        if (g * 8 >= nc) break;
                        uint4 o;
                        uint32_t* ou = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                        for (int e = 0; e < 4; e++) {
                            const int co = cc + g * 8 + 2 * e;
                            ou[e] = pack_half2(apply_act(v[g * 8 + 2 * e] + bias_s[co], p.act),
                                               apply_act(v[g * 8 + 2 * e + 1] + bias_s[co + 1], p.act));
                        }
                        const int g8 = (cc >> 3) + g;
                        *reinterpret_cast<uint4*>(stage_out + m * 128 + (((g8 & 7) ^ (m & 7)) << 4)) = o;
                    }
                }
                tc_fence_before_sync();
                fence_proxy_async_smem();
                work_bar_sync();
                if (threadIdx.x == 0) {
                    tma_store_4d(&tmy, stage_out, 0, wo0, ho0, n0);
                    tma_store_commit();
                    tma_store_wait_read();
                }
                work_bar_sync();
            }
            if (!have) break;
            prev_t = t;
        }
        if (threadIdx.x == 0) tma_store_wait_read();
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) {
        if (abort_s) __nanosleep(20000);
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 128);
    }
}

struct Tile {
    int tw, th, tn;
};

Tile pick_tile(int N, int Ho, int Wo) {
    Tile best{16, 8, 1};
    long long best_tiles = -1;
    for (int tw = 128; tw >= 2; tw >>= 1)
        for (int th = 128 / tw; th >= 1; th >>= 1) {
            const int tn = 128 / (tw * th);
            const long long tiles = static_cast<long long>((Wo + tw - 1) / tw) * ((Ho + th - 1) / th) * ((N + tn - 1) / tn);
            if (best_tiles < 0 || tiles < best_tiles) {
                best_tiles = tiles;
                best = Tile{tw, th, tn};
            }
        }
    return best;
}

int k_row(const ConvArgs& a) { return (a.kw * a.Cin + 7) / 8 * 8; }
int k_chunks(const ConvArgs& a) { return (a.kh * k_row(a) + 63) / 64; }
size_t smem_bytes(const ConvArgs& a) { return static_cast<size_t>(k_chunks(a)) * (2 * kPlane + 8192) + kPlane + 1024; }

}  // namespace

bool stem_tc_supported(const ConvArgs& a) {
    return a.groups == 1 && a.Cin >= 1 && a.Cin <= 4 && a.Cout % 8 == 0 && a.Cout >= 8 && a.Cout <= 64 && a.kh <= 7 &&
           a.kw <= 7 && (a.stride == 1 || a.stride == 2) && a.pool == 0 && a.res == nullptr && k_chunks(a) <= kMaxKChunks &&
           a.N >= 1 && a.Ho >= 1 && a.Wo >= 1;
}

int stem_tc_init() {
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(stem_tc_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(stem_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return cuda_fail(e);
        attr_set = true;
    }
    return DLF_OK;
}

int launch_stem_tc(const ConvArgs& a, int sm_count, int* status_dev, cudaStream_t s) {
    if (!stem_tc_supported(a)) return DLF_E_UNSUPPORTED;
    int rc = stem_tc_init();
    if (rc) return rc;
    StemParams p{};
    p.x = static_cast<const __half*>(a.x); p.w = static_cast<const __half*>(a.w); p.bias = a.bias; p.status = status_dev;
    p.N = a.N; p.H = a.H; p.W = a.W; p.Cin = a.Cin; p.Ho = a.Ho; p.Wo = a.Wo; p.Cout = a.Cout;
    p.kh = a.kh; p.kw = a.kw; p.stride = a.stride; p.pad = a.pad; p.act = a.act;
    p.KR = k_row(a);
    p.kchunks = k_chunks(a);
    p.BN = (a.Cout + 15) / 16 * 16;
    const Tile tl = pick_tile(a.N, a.Ho, a.Wo);
    p.TW = tl.tw; p.TH = tl.th; p.TN = tl.tn;
    p.tiles_w = (a.Wo + tl.tw - 1) / tl.tw;
    p.tiles_h = (a.Ho + tl.th - 1) / tl.th;
    p.tiles_n = (a.N + tl.tn - 1) / tl.tn;
    const long long n_work = static_cast<long long>(p.tiles_w) * p.tiles_h * p.tiles_n;
    if (n_work > 0x7fffffffLL) return DLF_E_UNSUPPORTED;
    p.n_work = static_cast<int>(n_work);
    CUtensorMap tmy;
    {
        const uint64_t dims[4] = {static_cast<uint64_t>(a.Cout), static_cast<uint64_t>(a.Wo), static_cast<uint64_t>(a.Ho),
                                  static_cast<uint64_t>(a.N)};
        const uint64_t strides[3] = {static_cast<uint64_t>(a.Cout) * 2, static_cast<uint64_t>(a.Wo) * a.Cout * 2,
                                     static_cast<uint64_t>(a.Ho) * a.Wo * a.Cout * 2};
        const uint32_t box[4] = {64, static_cast<uint32_t>(tl.tw), static_cast<uint32_t>(tl.th), static_cast<uint32_t>(tl.tn)};
        const uint32_t es[4] = {1, 1, 1, 1};
        rc = encode_tmap(&tmy, a.y, 4, dims, strides, box, es);
        if (rc) return rc;
    }
    const int grid = std::max(1, std::min(sm_count, p.n_work));
    const size_t smem = std::max<size_t>(smem_bytes(a), 120 * 1024);
    cudaError_t e = a.Cin == 3 ? launch_kernel(stem_tc_kernel<3>, grid, kThreads, smem, s, tmy, p)
                               : launch_kernel(stem_tc_kernel<0>, grid, kThreads, smem, s, tmy, p);
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

}  // namespace dlf
