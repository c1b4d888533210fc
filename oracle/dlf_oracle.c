/*
 * CPU checker for the fused-conv-group executor.  TEST INFRASTRUCTURE ONLY: nothing on
 * the product path may call into this file; it shares no code with the CUDA library.
 *
 * What it computes.  Layer fusion is an execution strategy that reaches exactly the
 * result of running the layers one after another (Sec. I: the fusion patterns are
 * "mathematically equivalent"; Sec. III-B: a fused layer's output is produced on chip
 * and reused at once).  So the checker is the plain definition of every layer, each
 * materialised in full:
 *   - direct convolution, the seven nested loops of Eq. 1's operation count
 *     (H_out, W_out, H_K, W_K, C_in, C_out, plus the batch), fp32 accumulator;
 *   - fully connected layer, the M*K*N loops of Eq. 2;
 *   - folded-BN bias, residual add, ReLU / ReLU6, 2x2 max-pool, 3x3 max-pool,
 *     global average pool (the fusable operator set of Sec. II-A).
 * The paper never states its precision; the reading taken here is fp16 storage with
 * fp32 arithmetic and ONE round-to-nearest-even to fp16 per layer, after bias,
 * residual and activation, whatever the fusion plan.
 *
 * Loop order inside one output element is fixed: kh, kw, ci ascending, accumulator
 * starting at +0, taps outside the image skipped (zero padding).  Products of two fp16
 * values are exact in fp32, so a fused multiply-add and a multiply followed by an add
 * round identically; the file is built with -ffp-contract=off anyway.
 *
 * OpenMP only spreads independent output rows over threads; it never splits a sum.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_ACT_NONE = 0, ORC_ACT_RELU = 1, ORC_ACT_RELU6 = 2 };

/* ---- IEEE binary16 <-> binary32, written from the format definition ---------------- */

float orc_h2f(uint16_t h) {
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t exp = (h >> 10) & 0x1Fu;
    uint32_t man = h & 0x3FFu;
    uint32_t bits;
    if (exp == 0) {
        if (man == 0) {
            bits = sign;
        } else { /* subnormal: value = man * 2^-24 */
            int e = -1;
            do { man <<= 1; e++; } while (!(man & 0x400u));
            bits = sign | ((uint32_t)(127 - 15 - e) << 23) | ((man & 0x3FFu) << 13);
        }
    } else if (exp == 31) {
        bits = sign | 0x7F800000u | (man << 13);
    } else {
        bits = sign | ((exp + 127 - 15) << 23) | (man << 13);
    }
    float f;
    memcpy(&f, &bits, 4);
    return f;
}

uint16_t orc_f2h(float f) {
    uint32_t x;
    memcpy(&x, &f, 4);
    uint16_t sign = (uint16_t)((x >> 16) & 0x8000u);
    uint32_t absx = x & 0x7FFFFFFFu;
    if (absx >= 0x7F800000u) /* inf / nan */
        return (uint16_t)(sign | 0x7C00u | ((absx > 0x7F800000u) ? 0x200u : 0u));
    int32_t e = (int32_t)(absx >> 23) - 127; /* unbiased exponent */
    uint32_t m = (absx & 0x7FFFFFu) | 0x800000u; /* 24-bit significand */
    if (e >= 16) return (uint16_t)(sign | 0x7C00u); /* beyond the largest finite */
    int shift; /* bits dropped from the 24-bit significand */
    uint32_t hexp;
    if (e >= -14) { shift = 13; hexp = (uint32_t)(e + 15); }
    else { shift = 13 + (-14 - e); hexp = 0; if (shift > 25) return sign; }
    uint32_t kept = m >> shift;
    uint32_t rem = m & ((1u << shift) - 1u);
    uint32_t halfway = 1u << (shift - 1);
    if (rem > halfway || (rem == halfway && (kept & 1u))) kept++;
    /* normal: kept has the hidden bit at 0x400, adding hexp-1 folds a carry into the exponent */
    uint32_t out = (hexp ? ((hexp - 1u) << 10) : 0u) + kept;
    if (out >= 0x7C00u) out = 0x7C00u;
    return (uint16_t)(sign | out);
}

void orc_h2f_array(const uint16_t* h, float* f, int64_t n) {
    for (int64_t i = 0; i < n; i++) f[i] = orc_h2f(h[i]);
}
void orc_f2h_array(const float* f, uint16_t* h, int64_t n) {
    for (int64_t i = 0; i < n; i++) h[i] = orc_f2h(f[i]);
}

static float activate(float v, int act) {
    if (act == ORC_ACT_RELU) return v > 0.0f ? v : 0.0f;
    if (act == ORC_ACT_RELU6) { v = v > 0.0f ? v : 0.0f; return v < 6.0f ? v : 6.0f; }
    return v;
}

int orc_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Convolution layer (dense, grouped or depthwise) with bias, optional residual, activation,
 * fp16 rounding and optional 2x2/2 max-pool.
 *   x   [N][H][W][Cin]            fp16
 *   w   [Cout][kh][kw][Cin/groups] fp16
 *   res [N][Ho][Wo][Cout]         fp16 or NULL (added before the activation)
 *   y   [N][Ho][Wo][Cout], or [N][Ho/2][Wo/2][Cout] when pool == 2
 * Ho = (H + 2 pad - kh) / stride + 1 (floor), same for Wo.  Returns 0, or -1 on bad sizes.
 */
int orc_conv2d(const uint16_t* x, int N, int H, int W, int Cin, const uint16_t* w,
               const float* bias, int Cout, int kh, int kw, int stride, int pad, int groups,
               const uint16_t* res, int act, int pool, uint16_t* y, int nthreads) {
    if (N < 0 || H <= 0 || W <= 0 || Cin <= 0 || Cout <= 0 || kh <= 0 || kw <= 0 || stride <= 0 ||
        pad < 0 || groups <= 0 || Cin % groups || Cout % groups || (pool != 0 && pool != 2))
        return -1;
    const int Ho = (H + 2 * pad - kh) / stride + 1, Wo = (W + 2 * pad - kw) / stride + 1;
    if (Ho <= 0 || Wo <= 0) return -1;
    const int cg = Cin / groups, og = Cout / groups;
    const int Hp = pool ? Ho / 2 : Ho, Wp = pool ? Wo / 2 : Wo;
    (void)nthreads;
#ifdef _OPENMP
    if (nthreads <= 0) nthreads = omp_get_max_threads();
#pragma omp parallel for collapse(2) schedule(dynamic, 1) num_threads(nthreads)
#endif
    for (int n = 0; n < N; n++) {
        for (int hp = 0; hp < Hp; hp++) {
            for (int wp = 0; wp < Wp; wp++) {
                for (int co = 0; co < Cout; co++) {
                    const int g = co / og;
                    float best = 0.0f;
                    const int win = pool ? 2 : 1;
                    for (int dy = 0; dy < win; dy++) {
                        for (int dx = 0; dx < win; dx++) {
                            const int ho = hp * win + dy, wo = wp * win + dx;
                            float acc = 0.0f;
                            for (int r = 0; r < kh; r++) {
                                const int hi = ho * stride - pad + r;
                                if (hi < 0 || hi >= H) continue;
                                for (int s = 0; s < kw; s++) {
                                    const int wi = wo * stride - pad + s;
                                    if (wi < 0 || wi >= W) continue;
                                    const uint16_t* xp = x + (((int64_t)n * H + hi) * W + wi) * Cin + (int64_t)g * cg;
                                    const uint16_t* wq = w + (((int64_t)co * kh + r) * kw + s) * cg;
                                    for (int ci = 0; ci < cg; ci++)
                                        acc = acc + orc_h2f(xp[ci]) * orc_h2f(wq[ci]);
                                }
                            }
                            float v = acc + bias[co];
                            if (res) v = v + orc_h2f(res[(((int64_t)n * Ho + ho) * Wo + wo) * Cout + co]);
                            v = orc_h2f(orc_f2h(activate(v, act)));
                            if ((dy == 0 && dx == 0) || v > best) best = v;
                        }
                    }
                    y[(((int64_t)n * Hp + hp) * Wp + wp) * Cout + co] = orc_f2h(best);
                }
            }
        }
    }
    return 0;
}

/* Fully connected layer: y[n][o] = act(sum_k x[n][k] w[o][k] + bias[o]), k ascending. */
int orc_fc(const uint16_t* x, int N, int K, const uint16_t* w, const float* bias, int M, int act,
           uint16_t* y, int nthreads) {
    if (N < 0 || K <= 0 || M <= 0) return -1;
    (void)nthreads;
#ifdef _OPENMP
    if (nthreads <= 0) nthreads = omp_get_max_threads();
#pragma omp parallel for schedule(static) num_threads(nthreads)
#endif
    for (int o = 0; o < M; o++) {
        for (int n = 0; n < N; n++) {
            float acc = 0.0f;
            const uint16_t* xp = x + (int64_t)n * K;
            const uint16_t* wq = w + (int64_t)o * K;
            for (int k = 0; k < K; k++) acc = acc + orc_h2f(xp[k]) * orc_h2f(wq[k]);
            y[(int64_t)n * M + o] = orc_f2h(activate(acc + bias[o], act));
        }
    }
    return 0;
}

/* Max-pool k x k, given stride and padding; taps outside the image are ignored. */
int orc_maxpool(const uint16_t* x, int N, int H, int W, int C, int k, int stride, int pad,
                uint16_t* y) {
    if (N < 0 || H <= 0 || W <= 0 || C <= 0 || k <= 0 || stride <= 0 || pad < 0 || pad >= k) return -1;
    const int Ho = (H + 2 * pad - k) / stride + 1, Wo = (W + 2 * pad - k) / stride + 1;
    if (Ho <= 0 || Wo <= 0) return -1;
    for (int n = 0; n < N; n++)
        for (int ho = 0; ho < Ho; ho++)
            for (int wo = 0; wo < Wo; wo++)
                for (int c = 0; c < C; c++) {
                    float best = -INFINITY;
                    for (int r = 0; r < k; r++) {
                        const int hi = ho * stride - pad + r;
                        if (hi < 0 || hi >= H) continue;
                        for (int s = 0; s < k; s++) {
                            const int wi = wo * stride - pad + s;
                            if (wi < 0 || wi >= W) continue;
                            const float v = orc_h2f(x[(((int64_t)n * H + hi) * W + wi) * C + c]);
                            if (v > best) best = v;
                        }
                    }
                    y[(((int64_t)n * Ho + ho) * Wo + wo) * C + c] = orc_f2h(best);
                }
    return 0;
}

/* Global average pool: fp32 sum over (h, w) ascending, times 1/(H*W) in fp32, one rounding. */
int orc_gavgpool(const uint16_t* x, int N, int H, int W, int C, uint16_t* y) {
    if (N < 0 || H <= 0 || W <= 0 || C <= 0) return -1;
    const float inv = 1.0f / (float)(H * W);
    for (int n = 0; n < N; n++)
        for (int c = 0; c < C; c++) {
            float acc = 0.0f;
            for (int h = 0; h < H; h++)
                for (int w2 = 0; w2 < W; w2++)
                    acc = acc + orc_h2f(x[(((int64_t)n * H + h) * W + w2) * C + c]);
            y[(int64_t)n * C + c] = orc_f2h(acc * inv);
        }
    return 0;
}
