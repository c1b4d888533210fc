// CUDA-core kernels for the layers that are bound by memory traffic or too narrow for the
// tensor cores: direct convolution for tiny channel counts (the C = 3 stems), depthwise 3x3,
// max / global-average pooling and the weight-streaming fully connected layer.  All use 128-bit
// accesses along the channel dimension of the NHWC tensors, fp32 arithmetic and a single
// round-to-nearest-even to fp16 per layer.  Grids are sized from the SM-count knob and loop over
// the work with a grid stride.
#include <cuda_fp16.h>

#include <algorithm>

#include "internal.h"
#include "ptx.cuh"

namespace dlf {

namespace {

constexpr int kBlocksPerSm = 8;

inline int grid_for(long long work_blocks, int sm_count) {
    long long cap = static_cast<long long>(sm_count) * kBlocksPerSm;
    long long g = work_blocks < cap ? work_blocks : cap;
    return static_cast<int>(g < 1 ? 1 : g);
}

// ---- direct convolution ---------------------------------------------------------------------------
// One thread = one output pixel (after the optional 2x2 pool) x 16 output channels.  The weights
// of the block's 16 channels are staged in shared memory as fp32, one (tap, 64-channel) slab at
// a time, and read as broadcasts.  Summation order is (kh, kw, ci) ascending in fp32.
constexpr int kDirCo = 16;
constexpr int kDirCi = 64;

__global__ void __launch_bounds__(128) conv_direct_kernel(ConvArgs a, long long n_pix, int co_blocks) {
    __shared__ float wsm[kDirCi][kDirCo];
    const __half* x = static_cast<const __half*>(a.x);
    const __half* w = static_cast<const __half*>(a.w);
    const __half* res = static_cast<const __half*>(a.res);
    __half* y = static_cast<__half*>(a.y);
    const int win = a.pool ? 2 : 1;
    const int Hp = a.Ho / win, Wp = a.Wo / win;
    const int cg = a.Cin / a.groups, og = a.Cout / a.groups;
    const long long pix_blocks = (n_pix + blockDim.x - 1) / blockDim.x;
    const long long total = pix_blocks * co_blocks;
    for (long long blk = blockIdx.x; blk < total; blk += gridDim.x) {
        const int cb = static_cast<int>(blk % co_blocks);
        const long long p = (blk / co_blocks) * blockDim.x + threadIdx.x;
        const int co0 = cb * kDirCo;
        const int g = co0 / og;  // a block of 16 channels never straddles groups (checked on host)
        const bool live = p < n_pix;
        int n = 0, hp = 0, wp = 0;
        if (live) {
            wp = static_cast<int>(p % Wp);
            hp = static_cast<int>((p / Wp) % Hp);
            n = static_cast<int>(p / (static_cast<long long>(Wp) * Hp));
        }
        float best[kDirCo];
        for (int q = 0; q < win * win; q++) {
            const int ho = hp * win + q / win, wo = wp * win + q % win;
            float acc[kDirCo];
#pragma unroll
            for (int j = 0; j < kDirCo; j++) acc[j] = 0.0f;
            for (int r = 0; r < a.kh; r++) {
                for (int s = 0; s < a.kw; s++) {
                    const int hi = ho * a.stride - a.pad + r, wi = wo * a.stride - a.pad + s;
                    const bool inside = live && hi >= 0 && hi < a.H && wi >= 0 && wi < a.W;
                    const __half* xp = x + ((static_cast<long long>(n) * a.H + hi) * a.W + wi) * a.Cin + g * cg;
                    for (int c0 = 0; c0 < cg; c0 += kDirCi) {
                        const int cn = min(kDirCi, cg - c0);
                        __syncthreads();
                        for (int i = threadIdx.x; i < cn * kDirCo; i += blockDim.x) {
                            const int ci = i / kDirCo, j = i % kDirCo;
                            const int co = co0 + j;
                            wsm[ci][j] = co < a.Cout
                                             ? __half2float(w[((static_cast<long long>(co) * a.kh + r) * a.kw + s) * cg + c0 + ci])
                                             : 0.0f;
                        }
                        __syncthreads();
                        if (inside) {
                            for (int ci = 0; ci < cn; ci++) {
                                const float xv = __half2float(xp[c0 + ci]);
#pragma unroll
                                for (int j = 0; j < kDirCo; j++) acc[j] = fmaf(xv, wsm[ci][j], acc[j]);
                            }
                        }
                    }
                }
            }
            if (live) {
#pragma unroll
                for (int j = 0; j < kDirCo; j++) {
                    const int co = co0 + j;
                    if (co < a.Cout) {
                        float v = acc[j] + a.bias[co];
                        if (res) v += __half2float(res[((static_cast<long long>(n) * a.Ho + ho) * a.Wo + wo) * a.Cout + co]);
                        v = __half2float(__float2half_rn(apply_act(v, a.act)));
                        best[j] = (q == 0) ? v : fmaxf(best[j], v);
                    }
                }
            }
        }
        if (live) {
            __half* yp = y + ((static_cast<long long>(n) * Hp + hp) * Wp + wp) * a.Cout + co0;
#pragma unroll
            for (int j = 0; j < kDirCo; j++)
                if (co0 + j < a.Cout) yp[j] = __float2half_rn(best[j]);
        }
    }
}

// ---- depthwise 3x3 ------------------------------------------------------------------------------------
// One thread = 8 channels x a strip of kDwStrip output columns of one output row.  The thread's 72
// weights and 8 biases are converted to fp32 once (the launch makes the total thread count a
// multiple of C/8, so a thread keeps its channels over the whole grid-stride loop); every input
// vector of the strip's three rows is loaded once (128 bits), converted once and used by all the
// outputs it touches.  Lanes run over the channel vectors first, so a warp reads contiguous NHWC
// runs.  fp32 accumulation in (kh, kw) order, one rounding.
constexpr int kDwStrip = 4;

template <int STRIDE>
__global__ void __launch_bounds__(128) dw3x3_kernel(ConvArgs a, long long total, int strips) {
    constexpr int kCols = (kDwStrip - 1) * STRIDE + 3;  // input columns one strip reads per row
    const int c8n = a.Cout / 8;
    const long long tid = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    const long long nthreads = static_cast<long long>(gridDim.x) * blockDim.x;
    if (tid >= total) return;
    const int c0 = static_cast<int>(tid % c8n) * 8;
    float w[9][8], b[8];
    {
        __align__(16) __half wv[72];  // weights of channels c0..c0+7: 72 consecutive halves starting at c0*9
        const uint4* wp4 = reinterpret_cast<const uint4*>(static_cast<const __half*>(a.w) + static_cast<long long>(c0) * 9);
#pragma unroll
        for (int k = 0; k < 9; k++) reinterpret_cast<uint4*>(wv)[k] = __ldg(wp4 + k);
#pragma unroll
        for (int j = 0; j < 8; j++) {
            b[j] = __ldg(a.bias + c0 + j);
#pragma unroll
            for (int t = 0; t < 9; t++) w[t][j] = __half2float(wv[j * 9 + t]);
        }
    }
    const __half2 lo = __float2half2_rn(a.act >= 1 ? 0.0f : -INFINITY), hi = __float2half2_rn(a.act == 2 ? 6.0f : INFINITY);   // applied to rounded pairs
    const __half* x = static_cast<const __half*>(a.x);
    const __half* res = static_cast<const __half*>(a.res);
    __half* y = static_cast<__half*>(a.y);
    for (long long i = tid; i < total; i += nthreads) {
        long long p = i / c8n;
        const int strip = static_cast<int>(p % strips);
        p /= strips;
        const int ho = static_cast<int>(p % a.Ho);
        const int n = static_cast<int>(p / a.Ho);
        const int wo0 = strip * kDwStrip;
        const int wi0 = wo0 * STRIDE - a.pad;
        float acc[kDwStrip][8];
#pragma unroll
        for (int o = 0; o < kDwStrip; o++)
#pragma unroll
            for (int j = 0; j < 8; j++) acc[o][j] = 0.0f;
#pragma unroll
        for (int r = 0; r < 3; r++) {
            const int hi_ = ho * STRIDE - a.pad + r;
            const bool row_ok = hi_ >= 0 && hi_ < a.H;
            const __half* row = x + ((static_cast<long long>(n) * a.H + min(max(hi_, 0), a.H - 1)) * a.W) * a.Cin + c0;
            // all loads of the row first, from clamped (always valid) addresses and without branches, so
            // that they are in flight together; columns outside the image are zeroed afterwards
            uint4 xv[kCols];
#pragma unroll
            for (int j = 0; j < kCols; j++)
                xv[j] = __ldg(reinterpret_cast<const uint4*>(row + static_cast<long long>(min(max(wi0 + j, 0), a.W - 1)) * a.Cin));
#pragma unroll
            for (int j = 0; j < kCols; j++) {
                const int wi = wi0 + j;
                // a column outside the image contributes zeros: the vector is cleared with four selects (a multiply
                // by 0 / 1 per element doubled the load on the FMA pipe, which is what bounds this kernel)
                if (!(row_ok && wi >= 0 && wi < a.W)) xv[j] = make_uint4(0u, 0u, 0u, 0u);
                const __half2* xh = reinterpret_cast<const __half2*>(&xv[j]);
                float xf[8];
#pragma unroll
                for (int e = 0; e < 4; e++) {
                    const float2 f = __half22float2(xh[e]);
                    xf[2 * e] = f.x;
                    xf[2 * e + 1] = f.y;
                }
#pragma unroll
                for (int o = 0; o < kDwStrip; o++) {
                    const int s = j - o * STRIDE;  // tap column of output o that reads input column j
                    if (s >= 0 && s < 3) {
#pragma unroll
                        for (int e = 0; e < 8; e++) acc[o][e] = fmaf(xf[e], w[r * 3 + s][e], acc[o][e]);
                    }
                }
            }
        }
#pragma unroll
        for (int o = 0; o < kDwStrip; o++) {
            const int wo = wo0 + o;
            if (wo >= a.Wo) break;
            const long long off = ((static_cast<long long>(n) * a.Ho + ho) * a.Wo + wo) * a.Cout + c0;
            float v[8];
#pragma unroll
            for (int e = 0; e < 8; e++) v[e] = acc[o][e] + b[e];
            if (res != nullptr) {
                const uint4 rv = __ldg(reinterpret_cast<const uint4*>(res + off));
                const __half2* rh = reinterpret_cast<const __half2*>(&rv);
#pragma unroll
                for (int e = 0; e < 4; e++) {
                    const float2 f = __half22float2(rh[e]);
                    v[2 * e] += f.x;
                    v[2 * e + 1] += f.y;
                }
            }
            uint4 outv;
            uint32_t* ou = reinterpret_cast<uint32_t*>(&outv);
#pragma unroll
            for (int e = 0; e < 4; e++)
                ou[e] = pack_half2_clamp(v[2 * e], v[2 * e + 1], lo, hi);
            *reinterpret_cast<uint4*>(y + off) = outv;
        }
    }
}

// ---- pooling ----------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) maxpool_kernel(const __half* x, __half* y, int N, int H, int W, int C, int k,
                                                      int stride, int pad, int Ho, int Wo, long long total) {
    const int c8n = C / 8;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int c8 = static_cast<int>(i % c8n);
        long long p = i / c8n;
        const int wo = static_cast<int>(p % Wo);
        p /= Wo;
        const int ho = static_cast<int>(p % Ho);
        const int n = static_cast<int>(p / Ho);
        __half2 best[4];
        const __half2 ninf = __half2half2(__ushort_as_half(0xFC00));
#pragma unroll
        for (int j = 0; j < 4; j++) best[j] = ninf;
        // clamped taps instead of skipped ones: a tap outside the image re-reads an in-range pixel of the
        // same window (the maximum is unchanged) and the loads carry no branches, so they overlap
        const int h_lo = max(ho * stride - pad, 0), h_hi = min(ho * stride - pad + k - 1, H - 1);
        const int w_lo = max(wo * stride - pad, 0), w_hi = min(wo * stride - pad + k - 1, W - 1);
        for (int r = 0; r < k; r++) {
            const int hi = min(max(ho * stride - pad + r, h_lo), h_hi);
#pragma unroll 3
            for (int s = 0; s < k; s++) {
                const int wi = min(max(wo * stride - pad + s, w_lo), w_hi);
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(x + ((static_cast<long long>(n) * H + hi) * W + wi) * C + c8 * 8));
                const __half2* vh = reinterpret_cast<const __half2*>(&v);
#pragma unroll
                for (int j = 0; j < 4; j++) best[j] = __hmax2(best[j], vh[j]);
            }
        }
        *reinterpret_cast<uint4*>(y + ((static_cast<long long>(n) * Ho + ho) * Wo + wo) * C + c8 * 8) =
            *reinterpret_cast<uint4*>(best);
    }
}

// fp32 sum over (h, w) ascending, times 1/(H*W), one rounding.
__global__ void __launch_bounds__(128) gavgpool_kernel(const __half* x, __half* y, int N, int HW, int C, long long total) {
    const int c8n = C / 8;
    const float inv = 1.0f / static_cast<float>(HW);
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int c8 = static_cast<int>(i % c8n);
        const int n = static_cast<int>(i / c8n);
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; j++) acc[j] = 0.0f;
        const __half* xp = x + static_cast<long long>(n) * HW * C + c8 * 8;
        for (int p = 0; p < HW; p++) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(xp + static_cast<long long>(p) * C));
            const __half* vh = reinterpret_cast<const __half*>(&v);
#pragma unroll
            for (int j = 0; j < 8; j++) acc[j] += __half2float(vh[j]);
        }
        uint4 o;
        uint32_t* ou = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
        for (int j = 0; j < 8; j += 2) ou[j / 2] = pack_half2(acc[j] * inv, acc[j + 1] * inv);
        *reinterpret_cast<uint4*>(y + static_cast<long long>(n) * C + c8 * 8) = o;
    }
}

// ---- fully connected --------------------------------------------------------------------------------------
// A block owns 8 output features and streams their weight rows once per batch tile of 8 images;
// threads stride over K in 128-bit pieces, accumulate 8x8 partial sums in fp32, then reduce.
constexpr int kFcFo = 8;
constexpr int kFcNb = 8;

__global__ void __launch_bounds__(256) fc_kernel(const __half* x, const __half* w, const float* bias, __half* y, int N,
                                                 int K, int M, int act, int o_blocks, int n_blocks) {
    __shared__ float red[8][kFcFo * kFcNb];
    const int k8n = K / 8;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int blk = blockIdx.x; blk < o_blocks * n_blocks; blk += gridDim.x) {
        const int o0 = (blk % o_blocks) * kFcFo, n0 = (blk / o_blocks) * kFcNb;
        float acc[kFcFo][kFcNb];
#pragma unroll
        for (int i = 0; i < kFcFo; i++)
#pragma unroll
            for (int j = 0; j < kFcNb; j++) acc[i][j] = 0.0f;
        for (int k8 = threadIdx.x; k8 < k8n; k8 += blockDim.x) {
            uint4 wv[kFcFo], xv[kFcNb];
#pragma unroll
            for (int i = 0; i < kFcFo; i++) {
                const int o = min(o0 + i, M - 1);
                wv[i] = __ldcs(reinterpret_cast<const uint4*>(w + static_cast<long long>(o) * K) + k8);
            }
#pragma unroll
            for (int j = 0; j < kFcNb; j++) {
                const int n = min(n0 + j, N - 1);
                xv[j] = __ldg(reinterpret_cast<const uint4*>(x + static_cast<long long>(n) * K) + k8);
            }
#pragma unroll
            for (int e = 0; e < 4; e++) {
                float2 xf[kFcNb];
#pragma unroll
                for (int j = 0; j < kFcNb; j++) xf[j] = __half22float2(reinterpret_cast<const __half2*>(&xv[j])[e]);
#pragma unroll
                for (int i = 0; i < kFcFo; i++) {
                    const float2 wf = __half22float2(reinterpret_cast<const __half2*>(&wv[i])[e]);
#pragma unroll
                    for (int j = 0; j < kFcNb; j++) {
                        acc[i][j] = fmaf(wf.x, xf[j].x, acc[i][j]);
                        acc[i][j] = fmaf(wf.y, xf[j].y, acc[i][j]);
                    }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < kFcFo; i++)
#pragma unroll
            for (int j = 0; j < kFcNb; j++) {
                float v = acc[i][j];
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
                if (lane == 0) red[warp][i * kFcNb + j] = v;
            }
        __syncthreads();
        if (threadIdx.x < kFcFo * kFcNb) {
            float v = 0.0f;
            for (int wq = 0; wq < 8; wq++) v += red[wq][threadIdx.x];
            const int o = o0 + threadIdx.x / kFcNb, n = n0 + threadIdx.x % kFcNb;
            if (o < M && n < N) y[static_cast<long long>(n) * M + o] = __float2half_rn(apply_act(v + bias[o], act));
        }
        __syncthreads();
    }
}

}  // namespace

int launch_conv_direct(const ConvArgs& a, int sm_count, cudaStream_t s) {
    const int og = a.Cout / a.groups;
    if (a.groups > 1 && og % kDirCo != 0) return DLF_E_UNSUPPORTED;
    const int win = a.pool ? 2 : 1;
    const long long n_pix = static_cast<long long>(a.N) * (a.Ho / win) * (a.Wo / win);
    const int co_blocks = (a.Cout + kDirCo - 1) / kDirCo;
    const long long blocks = (n_pix + 127) / 128 * co_blocks;
    if (blocks == 0) return DLF_OK;
    conv_direct_kernel<<<grid_for(blocks, sm_count), 128, 0, s>>>(a, n_pix, co_blocks);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

int launch_dw3x3(const ConvArgs& a, int sm_count, cudaStream_t s) {
    if (a.kh != 3 || a.kw != 3 || a.groups != a.Cin || a.Cin != a.Cout || a.Cin % 8 || a.pool) return DLF_E_UNSUPPORTED;
    if (a.stride != 1 && a.stride != 2) return DLF_E_UNSUPPORTED;
    const int c8n = a.Cout / 8;
    const int strips = (a.Wo + kDwStrip - 1) / kDwStrip;
    const long long total = static_cast<long long>(a.N) * a.Ho * strips * c8n;
    if (total == 0) return DLF_OK;
    // the total thread count is a multiple of C/8: a thread keeps its channels (and its weights)
    int step = c8n;
    for (int d = 2; d <= 128; d *= 2)
        if (step % 2 == 0) step /= 2;  // blocks needed for (blocks * 128) % c8n == 0: c8n / gcd(c8n, 128)
    // one resident wave of blocks: a thread converts its 72 weights once and then walks its strips (more blocks than fit
    // would each pay that prologue again, wave after wave).  A variant with four channels per thread (96 registers,
    // five blocks per SM instead of three) was measured 20 % slower: the index arithmetic per vector doubles.
    static int occ[2] = {0, 0};
    const int v = a.stride == 1 ? 0 : 1;
    if (occ[v] == 0) {
        cudaError_t e = v == 0 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ[v], dw3x3_kernel<1>, 128, 0)
                               : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ[v], dw3x3_kernel<2>, 128, 0);
        if (e != cudaSuccess || occ[v] < 1) occ[v] = 2;
    }
    long long blocks = std::min<long long>((total + 127) / 128, static_cast<long long>(sm_count) * occ[v]);
    blocks = std::max<long long>(step, blocks / step * step);
    if (a.stride == 1) dw3x3_kernel<1><<<static_cast<int>(blocks), 128, 0, s>>>(a, total, strips);
    else dw3x3_kernel<2><<<static_cast<int>(blocks), 128, 0, s>>>(a, total, strips);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

int launch_maxpool(const void* x, void* y, int N, int H, int W, int C, int k, int stride, int pad, int Ho, int Wo,
                   int sm_count, cudaStream_t s) {
    if (C % 8) return DLF_E_UNSUPPORTED;
    const long long total = static_cast<long long>(N) * Ho * Wo * (C / 8);
    if (total == 0) return DLF_OK;
    maxpool_kernel<<<grid_for((total + 255) / 256, sm_count), 256, 0, s>>>(
        static_cast<const __half*>(x), static_cast<__half*>(y), N, H, W, C, k, stride, pad, Ho, Wo, total);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

int launch_gavgpool(const void* x, void* y, int N, int H, int W, int C, int sm_count, cudaStream_t s) {
    if (C % 8) return DLF_E_UNSUPPORTED;
    const long long total = static_cast<long long>(N) * (C / 8);
    if (total == 0) return DLF_OK;
    gavgpool_kernel<<<grid_for((total + 127) / 128, sm_count), 128, 0, s>>>(
        static_cast<const __half*>(x), static_cast<__half*>(y), N, H * W, C, total);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

int launch_fc(const void* x, const void* w, const float* bias, void* y, int N, int K, int M, int act, int sm_count,
              cudaStream_t s) {
    if (K % 8) return DLF_E_UNSUPPORTED;
    if (N == 0) return DLF_OK;
    const int o_blocks = (M + kFcFo - 1) / kFcFo, n_blocks = (N + kFcNb - 1) / kFcNb;
    const int grid = grid_for(static_cast<long long>(o_blocks) * n_blocks, sm_count);
    fc_kernel<<<grid, 256, 0, s>>>(static_cast<const __half*>(x), static_cast<const __half*>(w), bias,
                                   static_cast<__half*>(y), N, K, M, act, o_blocks, n_blocks);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

// Self-test of the bounded waits: one CTA waits, with the waits' own routine, at a barrier that nothing ever arrives at.
// The wait has to give up after `limit_ns`, record its code in the status word and let the kernel end normally.
__global__ void stall_kernel(int* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_s;
    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(&bar, 1);
        fence_barrier_init();
    }
    __syncthreads();
    mbar_wait(&bar, 0u, &abort_s, status, 0xd00, limit_ns);
}

int launch_stall(int* status_dev, unsigned long long limit_ns, cudaStream_t s) {
    stall_kernel<<<1, 64, 0, s>>>(status_dev, limit_ns);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

}  // namespace dlf
