// First-layer ("stem") convolution on the tensor cores: C_in <= 4 (the RGB input), kernel up to
// 7x7, stride 1 or 2, up to 64 output channels, bias + activation.
//
// With three input channels a tap is only 6 bytes wide, far below what TMA can address (16-byte
// strides) or a UMMA K step can use, so the implicit-GEMM operand is built in shared memory by the
// CTA's own threads: for output pixel m and kernel row r the kw * C_in input values are contiguous
// in NHWC memory; they go (zero outside the image) into K positions r*KR .. r*KR+kw*C_in-1 of row m
// of a 128-byte-swizzled A tile (KR = kw*C_in rounded up to 8, K = kh*KR rounded up to 64).  The
// input patch under a tile of output pixels is a few KB, the A tile built from it 10x that, so the
// patch is first staged in shared memory (one pass of 2-byte loads, prefetched a tile ahead into
// registers) and the A rows are then cut out of it with 4-byte shared loads, a 16-bit funnel shift
// where a row starts on an odd half, and 16-byte swizzled stores.  The positions between kw*C_in
// and KR receive the next pixels of the patch (finite values) and meet zero weights.
// The weights are laid out the same way once per CTA.  One thread then issues the UMMAs
// (M = 128 pixels, N = C_out, K) into one of two TMEM accumulators while the same eight warps
// build the next tile and drain the previous one (bias, activation, fp16 rounding, staging tile,
// TMA store).  Eq. 1 counts kh*kw*C_in*C_out MACs per output pixel; the padded K positions hold
// zeros on both operands.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <type_traits>

#include "internal.h"
#include "ptx.cuh"

namespace dlf {

namespace {

constexpr int kWorkWarps = 8;                 // warps 0..7 build A tiles and run the epilogue
constexpr int kMmaWarp = kWorkWarps;          // warp 8 issues the UMMAs and owns the TMEM allocation
constexpr int kThreads = 32 * (kWorkWarps + 1);
constexpr int kPlane = 128 * 128;             // one 64-wide K chunk of the A tile
constexpr int kMaxKChunks = 4;
constexpr int kMaxDynSmem = 232448 - 1024;   // the 227 KB per CTA less the kernel's static shared memory

struct StemParams {
    const __half* x;
    const __half* w;
    const float* bias;
    int* status;
    int N, H, W, Cin, Ho, Wo, Cout;
    int kh, kw, stride, pad, act;
    int KR, kchunks, BN;
    int TW, TH, TN, tiles_w, tiles_h, tiles_n, n_work;
    int lw, lh;                 // log2 of TW, TH (tile extents are powers of two)
    int rows_img, pitch_w;      // patch rows per image of the tile, 32-bit words per patch row
    int patch_words, patch_off; // words of one patch buffer; byte offset of the two patch buffers
};

constexpr int kPatchRegs = 8;                 // prefetched patch words per thread
constexpr int kMaxPatchWords = kPatchRegs * 32 * kWorkWarps;

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
    // layout: A[2][kchunks][128 x 128 B] | B[kchunks][64 x 128 B] | staging [2][128 x 128 B] | patch [2]
    const int a_bytes = p.kchunks * kPlane;
    uint8_t* bsm = sbase + 2 * a_bytes;
    uint8_t* stage_out = bsm + p.kchunks * 8192;
    uint32_t* patch = reinterpret_cast<uint32_t*>(sbase + p.patch_off);   // [2][patch_words]
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
    for (int i = threadIdx.x; i < 2 * p.patch_words; i += kThreads) patch[i] = 0u;
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
        const int q = warp & 3, half = warp >> 2;
        const uint32_t* x32 = reinterpret_cast<const uint32_t*>(p.x);
        const int row_halves = p.W * cin;
        // Patch word `widx` of a tile sits at (image nl, patch row y, word wI); that split does not
        // depend on the tile, so each thread keeps it, and the row's offset in the tensor, for its
        // kPatchRegs words.
        uint32_t meta[kPatchRegs];
        int rel[kPatchRegs];
#pragma unroll
        for (int i = 0; i < kPatchRegs; i++) {
            const int widx = min(static_cast<int>(threadIdx.x) + i * 32 * kWorkWarps, p.patch_words - 1);
            const int prow = widx / p.pitch_w, wI = widx - prow * p.pitch_w;
            const int nl = prow / p.rows_img, y = prow - nl * p.rows_img;
            meta[i] = static_cast<uint32_t>(wI) | (static_cast<uint32_t>(y) << 12) | (static_cast<uint32_t>(nl) << 22);
            rel[i] = (nl * p.H + y) * row_halves;
        }
        // A patch row is kept as the aligned 32-bit words of the tensor that cover it, so a row whose
        // first element sits on an odd half starts one half into its buffer row.  One unconditional
        // clamped load per word, all in flight together; `okm` keeps which halves lie inside the
        // image and the batch (the others become zero when the words are stored).
        // first output pixel of a tile; decoded once per tile (three divisions) and handed from the patch fetch to the
        // build to the drain
        struct TileOrigin { int wo0, ho0, n0; };
        auto decode = [&](int t) {
            TileOrigin o;
            int mt = t;
            o.wo0 = (mt % p.tiles_w) * p.TW;
            mt /= p.tiles_w;
            o.ho0 = (mt % p.tiles_h) * p.TH;
            o.n0 = (mt / p.tiles_h) * p.TN;
            return o;
        };
        auto load_patch = [&](const TileOrigin& to, uint32_t (&pw)[kPatchRegs], uint32_t& okm) {
            const int wo0 = to.wo0, ho0 = to.ho0, n0 = to.n0;
            const int wi0 = wo0 * p.stride - p.pad, hi0 = ho0 * p.stride - p.pad;
            const int tile_base = ((n0 * p.H + hi0) * p.W + wi0) * cin;
            const int h_lo = max(0, -wi0) * cin, h_hi = (p.W - wi0) * cin;   // halves of a patch row inside the image
            okm = 0u;
#pragma unroll
            for (int i = 0; i < kPatchRegs; i++) {
                if (i * 32 * kWorkWarps >= p.patch_words) break;   // (uniform) a small patch needs only the first few passes
                const int wI = meta[i] & 0xFFF, y = (meta[i] >> 12) & 0x3FF, nl = meta[i] >> 22;
                const int n = n0 + nl, hi_row = hi0 + y;
                const bool row_ok = n < p.N && hi_row >= 0 && hi_row < p.H;
                const int g_row = tile_base + rel[i];                // first half of the patch row in the tensor
                const int h0 = 2 * wI - (g_row & 1);                 // this word's halves, counted from there
                const bool ok0 = row_ok && h0 >= h_lo && h0 < h_hi, ok1 = row_ok && h0 + 1 >= h_lo && h0 + 1 < h_hi;
                const int gw = ((g_row & ~1) >> 1) + wI;
                pw[i] = __ldg(x32 + ((ok0 || ok1) ? gw : 0));
                okm |= ((ok0 ? 1u : 0u) | (ok1 ? 2u : 0u)) << (2 * i);
            }
        };
        auto store_patch = [&](uint32_t* dst, const uint32_t (&pw)[kPatchRegs], uint32_t okm) {
#pragma unroll
            for (int i = 0; i < kPatchRegs; i++) {
                if (i * 32 * kWorkWarps >= p.patch_words) break;
                const int widx = threadIdx.x + i * 32 * kWorkWarps;
                const uint32_t m = ((okm >> (2 * i)) & 1u ? 0x0000FFFFu : 0u) | ((okm >> (2 * i)) & 2u ? 0xFFFF0000u : 0u);
                if (widx < p.patch_words) dst[widx] = pw[i] & m;
            }
        };
        // rows of the A tile from the staged patch, CH 16-byte chunks per kernel row
        auto build_rows = [&](auto ch_tag, const TileOrigin& to, uint8_t* abuf, const uint32_t* pbuf) {
            constexpr int CH = decltype(ch_tag)::value;
            const int wo0 = to.wo0, ho0 = to.ho0, n0 = to.n0;
            const int tile_base = ((n0 * p.H + ho0 * p.stride - p.pad) * p.W + wo0 * p.stride - p.pad) * cin;
            const int sc = p.stride * cin;
#pragma unroll 2
            for (int item = threadIdx.x; item < 128 * p.kh; item += 32 * kWorkWarps) {
                const int m = item & 127, r = item >> 7;
                const int tx = m & (p.TW - 1), ty = (m >> p.lw) & (p.TH - 1), nl = m >> (p.lw + p.lh);
                const int yrow = ty * p.stride + r;
                const int off = ((tile_base + (nl * p.H + yrow) * row_halves) & 1) + tx * sc;   // first half of the K slice
                const uint32_t* src = pbuf + (nl * p.rows_img + yrow) * p.pitch_w + (off >> 1);
                const uint32_t sh = (off & 1) * 16;
                uint32_t w[4 * CH + 1];
#pragma unroll
                for (int i = 0; i <= 4 * CH; i++) w[i] = src[i];
#pragma unroll
                for (int ck = 0; ck < CH; ck++) {
                    uint4 o;
                    o.x = __funnelshift_r(w[4 * ck], w[4 * ck + 1], sh);
                    o.y = __funnelshift_r(w[4 * ck + 1], w[4 * ck + 2], sh);
                    o.z = __funnelshift_r(w[4 * ck + 2], w[4 * ck + 3], sh);
                    o.w = __funnelshift_r(w[4 * ck + 3], w[4 * ck + 4], sh);
                    const int kchunk = r * CH + ck;  // 16-byte chunk index along K
                    *reinterpret_cast<uint4*>(abuf + (kchunk >> 3) * kPlane + m * 128 + (((kchunk & 7) ^ (m & 7)) << 4)) = o;
                }
            }
        };
        uint32_t pw[kPatchRegs];
        uint32_t pok = 0u;
        TileOrigin cur = decode(blockIdx.x), next = cur, prev = cur;
        if (static_cast<int>(blockIdx.x) < p.n_work) {
            load_patch(cur, pw, pok);
            store_patch(patch, pw, pok);
        }
        // the activation as a clamp: none (-inf, inf), ReLU [0, inf), ReLU6 [0, 6]
        // (applied to the rounded pair: rounding is monotone and 0 and 6 are fp16 values, so clamping after the rounding gives
        // the same bits as before it, at one instruction per two values)
        const __half2 act_lo = __float2half2_rn(p.act == DLF_ACT_NONE ? -INFINITY : 0.0f), act_hi = __float2half2_rn(p.act == DLF_ACT_RELU6 ? 6.0f : INFINITY);
        // this warp's 32 output channels per pass of the epilogue keep their bias in registers
        float breg[32];
#pragma unroll
        for (int e = 0; e < 32; e++) breg[e] = bias_s[(half * 32 + e) & 63];
        work_bar_sync();
        DLF_TRACE_DECL(tacc, tmark);
        uint32_t j = 0;
        bool ok = true;
        int prev_t = -1;
        // software pipeline: fetch the patch of tile j+1, build tile j, then drain tile j-1 while the
        // tensor core works on tile j
        for (int t = blockIdx.x;; t += gridDim.x, j++) {
            const bool have = t < p.n_work;
            const bool have_next = have && t + static_cast<int>(gridDim.x) < p.n_work;
            DLF_TRACE_ACC(tacc, 0, tmark);
            if (have_next) {
                next = decode(t + gridDim.x);
                load_patch(next, pw, pok);
            }
            DLF_TRACE_ACC(tacc, 1, tmark);
            if (have) {
                uint8_t* abuf = sbase + (j & 1u) * a_bytes;
                const uint32_t* pbuf = patch + (j & 1u) * p.patch_words;
                switch (p.KR >> 3) {
                    case 1: build_rows(std::integral_constant<int, 1>{}, cur, abuf, pbuf); break;
                    case 2: build_rows(std::integral_constant<int, 2>{}, cur, abuf, pbuf); break;
                    case 3: build_rows(std::integral_constant<int, 3>{}, cur, abuf, pbuf); break;
                    default: build_rows(std::integral_constant<int, 4>{}, cur, abuf, pbuf); break;
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&a_full_bar[j & 1u]);
                DLF_TRACE_ACC(tacc, 2, tmark);
            }
            if (prev_t >= 0) {
                const uint32_t jb = j - 1, b = jb & 1u;
                ok = mbar_wait(&t_full_bar[b], (jb >> 1) & 1u, abort_flag, p.status, 0xA00 | (blockIdx.x << 12));
                DLF_TRACE_ACC(tacc, 3, tmark);
                if (!ok) break;
                tc_fence_after_sync();
                const int wo0 = prev.wo0, ho0 = prev.ho0, n0 = prev.n0;
                const int m = q * 32 + lane;
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + b * 64u;
                uint8_t* sout = stage_out + b * kPlane;   // its previous store was waited for before the last barrier
                const int cc = half * 32;
                if (cc < p.BN) {
                    float v[32];
                    const int nc = min(32, p.BN - cc);
                    if (nc == 32) tmem_ld32(taddr + cc, v);
                    else tmem_ld16(taddr + cc, v);
#pragma unroll
                    for (int g = 0; g < 4; g++) {
                        if (g * 8 >= nc) break;
                        uint4 o;
                        uint32_t* ou = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                        for (int e = 0; e < 4; e++)
                        {
                            const __half2 hv = __hmin2(__hmax2(__floats2half2_rn(v[g * 8 + 2 * e] + breg[g * 8 + 2 * e], v[g * 8 + 2 * e + 1] + breg[g * 8 + 2 * e + 1]), act_lo), act_hi);
                            ou[e] = *reinterpret_cast<const uint32_t*>(&hv);
                        }
                        const int g8 = (cc >> 3) + g;
                        *reinterpret_cast<uint4*>(sout + m * 128 + (((g8 & 7) ^ (m & 7)) << 4)) = o;
                    }
                }
                tc_fence_before_sync();
                fence_proxy_async_smem();
                DLF_TRACE_ACC(tacc, 4, tmark);
                work_bar_sync();
                if (threadIdx.x == 0) {
                    tma_store_4d(&tmy, sout, 0, wo0, ho0, n0);
                    tma_store_commit();
                }
            }
            if (!have) break;
            prev_t = t;
            prev = cur;
            cur = next;
            DLF_TRACE_ACC(tacc, 5, tmark);
            if (have_next) store_patch(patch + ((j + 1) & 1u) * p.patch_words, pw, pok);
            // the staging buffer the next drain writes was read by the store before the newest one
            if (threadIdx.x == 0) tma_store_wait_read1();
            work_bar_sync();
            DLF_TRACE_ACC(tacc, 6, tmark);
        }
        DLF_TRACE_FLUSH(p.status, tacc);
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

int k_row(const ConvArgs& a) { return (a.kw * a.Cin + 7) / 8 * 8; }
int k_chunks(const ConvArgs& a) { return (a.kh * k_row(a) + 63) / 64; }

// 32-bit words of one input-patch row under a tile `tw` pixels wide: an odd first half, the last
// pixel's K slice and the word the funnel shift looks ahead
// The pitch is then padded (by up to 31 words) to the value for which the 32 lanes of a warp, which
// read the same word of 32 consecutive output pixels' K slices, spread over the most banks.
int patch_pitch_words(const ConvArgs& a, int tw, int th) {
    const int need = (((tw - 1) * a.stride * a.Cin + k_row(a) + 4 + 7) / 8 * 8) / 2;
    const int rows_img = (th - 1) * a.stride + a.kh;
    int best = need, best_conf = 1 << 30;
    for (int pitch = need; pitch < need + 32; pitch++) {
        int worst = 0;
        for (int q = 0; q < 4 && q * 32 < 128; q++)
            for (int odd = 0; odd < 2; odd++) {
                int cnt[32] = {0};
                for (int lane = 0; lane < 32; lane++) {
                    const int m = q * 32 + lane, tx = m % tw, ty = (m / tw) % th, nl = m / (tw * th);
                    const int off = odd + tx * a.stride * a.Cin;
                    cnt[((nl * rows_img + ty * a.stride) * pitch + (off >> 1)) & 31]++;
                }
                int mx = 0;
                for (int b = 0; b < 32; b++) mx = std::max(mx, cnt[b]);
                worst = std::max(worst, mx);
            }
        if (worst < best_conf) {
            best_conf = worst;
            best = pitch;
        }
    }
    return best;
}
int patch_rows(const ConvArgs& a, int th) { return (th - 1) * a.stride + a.kh; }

// Fewest tiles of 128 output pixels (tw x th x tn, powers of two) whose input patch fits the
// prefetch registers; tw == 0 if none does.
Tile pick_tile(const ConvArgs& a) {
    const int N = a.N, Ho = a.Ho, Wo = a.Wo;
    Tile best{0, 0, 0};
    long long best_tiles = -1;
    for (int tw = 128; tw >= 1; tw >>= 1)
        for (int th = 128 / tw; th >= 1; th >>= 1) {
            const int tn = 128 / (tw * th);
            if (static_cast<long long>(tn) * patch_rows(a, th) * patch_pitch_words(a, tw, th) > kMaxPatchWords) continue;
            const long long tiles = static_cast<long long>((Wo + tw - 1) / tw) * ((Ho + th - 1) / th) * ((N + tn - 1) / tn);
            if (best_tiles < 0 || tiles < best_tiles) {
                best_tiles = tiles;
                best = Tile{tw, th, tn};
            }
        }
    return best;
}

// The patch is fetched as aligned 32-bit words indexed with 32-bit arithmetic: an even number of
// input elements (no word straddles the end of the tensor) below 2^31.
bool input_ok(const ConvArgs& a) {
    const long long total = static_cast<long long>(a.N) * a.H * a.W * a.Cin;
    return total % 2 == 0 && total + 2LL * 128 * a.H * a.W * a.Cin < 0x7fffffffLL;
}
size_t fixed_bytes(const ConvArgs& a) { return static_cast<size_t>(k_chunks(a)) * (2 * kPlane + 8192) + 2 * kPlane; }
size_t smem_bytes(const ConvArgs& a) { return fixed_bytes(a) + 2 * kMaxPatchWords * 4 + 1024; }

}  // namespace

bool stem_tc_supported(const ConvArgs& a) {
    return a.groups == 1 && a.Cin >= 1 && a.Cin <= 4 && a.Cout % 8 == 0 && a.Cout >= 8 && a.Cout <= 64 && a.kh <= 7 &&
           a.kw <= 7 && (a.stride == 1 || a.stride == 2) && a.pool == 0 && a.res == nullptr && k_chunks(a) <= kMaxKChunks &&
           a.N >= 1 && a.Ho >= 1 && a.Wo >= 1 && smem_bytes(a) <= static_cast<size_t>(kMaxDynSmem) && input_ok(a) && pick_tile(a).tw > 0;
}

int stem_tc_init() {
    static bool attr_set[kMaxDevices] = {};
    const int dev = current_device_slot();
    if (dev < 0) return DLF_E_UNSUPPORTED;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(stem_tc_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(stem_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
        if (e != cudaSuccess) return cuda_fail(e);
        attr_set[dev] = true;
    }
    return DLF_OK;
}

int launch_stem_tc(const ConvArgs& a, int sm_count, int* status_dev, cudaStream_t s) {
    if (!stem_tc_supported(a)) return DLF_E_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(a.x) & 3u) return DLF_E_INVALID_ARG;
    int rc = stem_tc_init();
    if (rc) return rc;
    StemParams p{};
    p.x = static_cast<const __half*>(a.x); p.w = static_cast<const __half*>(a.w); p.bias = a.bias; p.status = status_dev;
    p.N = a.N; p.H = a.H; p.W = a.W; p.Cin = a.Cin; p.Ho = a.Ho; p.Wo = a.Wo; p.Cout = a.Cout;
    p.kh = a.kh; p.kw = a.kw; p.stride = a.stride; p.pad = a.pad; p.act = a.act;
    p.KR = k_row(a);
    p.kchunks = k_chunks(a);
    p.BN = (a.Cout + 15) / 16 * 16;
    const Tile tl = pick_tile(a);
    p.TW = tl.tw; p.TH = tl.th; p.TN = tl.tn;
    for (p.lw = 0; (1 << p.lw) < tl.tw; p.lw++) {}
    for (p.lh = 0; (1 << p.lh) < tl.th; p.lh++) {}
    p.rows_img = patch_rows(a, tl.th);
    p.pitch_w = patch_pitch_words(a, tl.tw, tl.th);
    p.patch_words = tl.tn * p.rows_img * p.pitch_w;
    p.patch_off = static_cast<int>(fixed_bytes(a));
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
