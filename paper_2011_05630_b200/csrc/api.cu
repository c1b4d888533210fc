// Host side of the library: the layer list and its shape / operation-count inference (Eq. 1,
// Eq. 2), fusion plans (Algorithm 1's two output arrays) and their validation, the launcher that
// turns a plan into one kernel per group on a persistent grid of `sm_count` CTAs, timing, the
// auto-tuner (Eq. 5 + Algorithm 1) and the reduced brute-force search (Sec. V).
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <limits>
#include <new>
#include <vector>

#include "internal.h"

namespace dlf {

static thread_local int g_last_cuda_error = 0;
int g_use_pdl = 1;
int g_conv_row_mode = 1;

int cuda_fail(cudaError_t e) {
    g_last_cuda_error = static_cast<int>(e);
    cudaGetLastError();
    return DLF_E_CUDA;
}
int cuda_fail_drv(int e) {
    g_last_cuda_error = 100000 + e;
    return DLF_E_CUDA;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int encode_tmap(void* out_map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                const uint32_t* box, const uint32_t* elem_strides) {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr);
        if (e != cudaSuccess) return cuda_fail(e);
        if (qr != cudaDriverEntryPointSuccess || !p) return cuda_fail_drv(999);
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    cuuint64_t gd[5], gs[4];
    cuuint32_t bx[5], es[5];
    for (int i = 0; i < rank; i++) {
        gd[i] = dims[i];
        bx[i] = box[i];
        es[i] = elem_strides[i];
        if (i < rank - 1) gs[i] = strides_bytes[i];
    }
    CUresult r = fn(static_cast<CUtensorMap*>(out_map), CU_TENSOR_MAP_DATA_TYPE_FLOAT16, static_cast<cuuint32_t>(rank),
                    const_cast<void*>(base), gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail_drv(static_cast<int>(r));
    return DLF_OK;
}

enum Kind { K_CHAIN_TC, K_CONV_TC, K_CONV_DIRECT, K_DW, K_FC, K_MAXPOOL, K_GAVG, K_STEM_TC, K_MBCONV, K_CONV_SEQ, K_CONV_DUAL };
static const char* kKindName[] = {"chain_tc", "conv_tc", "conv_direct", "dw3x3", "fc", "maxpool", "gavgpool", "stem_tc", "mbconv_tc", "conv_seq", "conv_tc"};

struct Layer {
    dlf_layer_desc d;
    int64_t in[4], out[4];
    int ho_pre, wo_pre;  // before the fused pool
    int64_t ops_eq1, flops, w_elems;
    const void* w;
    const float* bias;
    size_t off, bytes;  // slot in the workspace
};

struct Group {
    int first, last, sms;
    Kind kind;
    ChainTiling tiling;
    MbconvTiling mb_tiling;
};

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct GraphCache {
    cudaGraphExec_t exec = nullptr;
    const void* in = nullptr;
    void* out = nullptr;
    void drop() {
        if (exec) cudaGraphExecDestroy(exec);
        exec = nullptr;
    }
};

}  // namespace dlf

using namespace dlf;

struct dlf_net {
    int N, H, W, C;
    std::vector<Layer> layers;
    std::vector<Group> plan;
    uint8_t* ws = nullptr;
    size_t ws_bytes = 0, ws_need = 0, in_off = 0, in_bytes = 0, status_off = 0, splitk_off = 0;
    int dev_sms = 0;
    int opt_no_tc = 0, opt_single_chain = 0, opt_graph = 1, opt_group_kernel = 0;
    const void* last_out = nullptr;
    // One CUDA graph per (input, output) pointer pair holds the whole plan; a second, instrumented
    // one records an event after every group for per-group timing.
    dlf::GraphCache graph, graph_timed;
    std::vector<cudaEvent_t> group_events;
    cudaStream_t capture_stream = nullptr;
    ~dlf_net();
};

namespace dlf {

// Split-K scratch at the end of a net's workspace: 64 KB of counters and 16 MB of fp32 partial tiles.
constexpr size_t kSplitKCounterBytes = 65536;
constexpr size_t kSplitKBytes = kSplitKCounterBytes + (16u << 20);

static bool is_param(const Layer& l) { return l.d.op == DLF_CONV || l.d.op == DLF_DWCONV || l.d.op == DLF_FC; }

static int query_sms(int* out) {
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    *out = sms;
    return DLF_OK;
}

// ---- structure of fusable chains ----------------------------------------------------------------
// Layers first..last can be ONE fused kernel only if they form a chain of dense stride-1
// size-keeping convolutions (1x1 or 3x3), each reading its predecessor, with pooling / residual
// on the last layer only and no intermediate map used anywhere else.  Pure function of the list.
static bool chain_layer_ok(const Layer& l) {
    const dlf_layer_desc& d = l.d;
    return d.op == DLF_CONV && d.groups == 1 && d.stride == 1 && d.kh == d.kw && (d.kh == 1 || d.kh == 3) &&
           d.pad == d.kh / 2 && chain_tc_layer_supported(d.cin, d.cout, d.kh);
}

static bool span_is_chain(const dlf_net* net, int first, int last) {
    if (last - first + 1 > kMaxChain) return false;
    const int n = static_cast<int>(net->layers.size());
    for (int i = first; i <= last; i++) {
        const Layer& l = net->layers[i];
        if (!chain_layer_ok(l)) return false;
        if (i > first && l.d.src != i - 1) return false;
        if (i < last && (l.d.pool != 0 || l.d.res_src != -2)) return false;
        if (i == last && l.d.res_src >= first) return false;
    }
    // no outside use of an intermediate map
    for (int j = first + 1; j < n; j++) {
        const dlf_layer_desc& d = net->layers[j].d;
        const int refs[2] = {d.src, d.res_src};
        for (int r : refs) {
            if (r < first || r >= last) continue;        // not an intermediate of this span
            if (j <= last && r == j - 1 && r == d.src) {  // the chain edge itself
                if (d.res_src == r) return false;
                continue;
            }
            return false;
        }
    }
    return true;
}

// ---- inverted-residual pattern ------------------------------------------------------------------------
// [1x1 conv (expansion), depthwise 3x3, 1x1 conv (projection)] or, without expansion, [depthwise 3x3,
// 1x1 conv]: each layer reads its predecessor, no pooling, a residual only on the projection and
// from outside the span, the maps between the layers used nowhere else.  `prefix` accepts the
// pattern's first layers (a block that may still grow into the pattern).
static bool pointwise_ok(const dlf_layer_desc& d) {
    return d.op == DLF_CONV && d.groups == 1 && d.kh == 1 && d.kw == 1 && d.stride == 1 && d.pad == 0 && d.pool == 0;
}
static bool depthwise_ok(const dlf_layer_desc& d) {
    return d.op == DLF_DWCONV && d.kh == 3 && d.kw == 3 && d.pad == 1 && (d.stride == 1 || d.stride == 2) && d.pool == 0 &&
           d.res_src == -2;
}
static bool span_is_mbconv(const dlf_net* net, int first, int last, bool prefix) {
    const int len = last - first + 1;
    if (len < 2 || len > 3) return false;
    const dlf_layer_desc& d0 = net->layers[first].d;
    const bool has_expand = d0.op == DLF_CONV;
    const int n_full = has_expand ? 3 : 2;
    if (len > n_full || (!prefix && len != n_full)) return false;
    int idx = first;
    if (has_expand) {
        if (!pointwise_ok(d0) || d0.res_src != -2) return false;
        idx++;
    }
    const dlf_layer_desc& dd = net->layers[idx].d;
    if (!depthwise_ok(dd) || (idx > first && dd.src != idx - 1)) return false;
    int hid = dd.cin, cout = 8;  // no projection yet (a prefix): nothing to check on its width
    if (idx < last) {
        const dlf_layer_desc& dp = net->layers[idx + 1].d;
        if (!pointwise_ok(dp) || dp.src != idx || dp.res_src >= first) return false;
        cout = dp.cout;
    }
    MbconvArgs a;
    std::memset(&a, 0, sizeof(a));
    a.N = 1; a.H = 8; a.W = 8;
    a.Cin = has_expand ? d0.cin : hid; a.hid = hid; a.Cout = cout; a.stride = dd.stride; a.has_expand = has_expand ? 1 : 0;
    if (!mbconv_supported(a)) return false;
    // the maps between the layers are used nowhere else
    const int n = static_cast<int>(net->layers.size());
    for (int j = first + 1; j < n; j++) {
        const dlf_layer_desc& d = net->layers[j].d;
        const int refs[2] = {d.src, d.res_src};
        for (int k = 0; k < 2; k++) {
            const int r = refs[k];
            if (r < first || r >= last) continue;
            if (k == 0 && j <= last && r == j - 1) continue;
            return false;
        }
    }
    return true;
}

static inline const uint8_t* slot(const dlf_net* net, int idx) {
    return net->ws ? net->ws + net->layers[idx].off : nullptr;
}

static ChainArgs chain_args(const dlf_net* net, int first, int last, const void* in_dev, void* out_dev) {
    ChainArgs a;
    std::memset(&a, 0, sizeof(a));
    a.n_layers = last - first + 1;
    const Layer& f = net->layers[first];
    const Layer& z = net->layers[last];
    a.x = f.d.src < 0 ? in_dev : slot(net, f.d.src);
    for (int i = first; i <= last; i++) {
        const Layer& l = net->layers[i];
        a.w[i - first] = l.w;
        a.bias[i - first] = l.bias;
        a.cin[i - first] = l.d.cin;
        a.cout[i - first] = l.d.cout;
        a.k[i - first] = l.d.kh;
        a.act[i - first] = l.d.act;
    }
    a.res = z.d.res_src == -2 ? nullptr : (z.d.res_src < 0 ? in_dev : slot(net, z.d.res_src));
    a.y = out_dev;
    a.N = static_cast<int>(f.in[0]);
    a.H = static_cast<int>(f.in[1]);
    a.W = static_cast<int>(f.in[2]);
    a.pool = z.d.pool;
    return a;
}

static ConvArgs conv_args(const dlf_net* net, int i, const void* in_dev, void* out_dev) {
    const Layer& l = net->layers[i];
    ConvArgs a;
    std::memset(&a, 0, sizeof(a));
    a.x = l.d.src < 0 ? in_dev : slot(net, l.d.src);
    a.w = l.w;
    a.bias = l.bias;
    a.res = l.d.res_src == -2 ? nullptr : (l.d.res_src < 0 ? in_dev : slot(net, l.d.res_src));
    a.y = out_dev;
    a.N = static_cast<int>(l.in[0]); a.H = static_cast<int>(l.in[1]); a.W = static_cast<int>(l.in[2]);
    a.Cin = l.d.cin; a.Ho = l.ho_pre; a.Wo = l.wo_pre; a.Cout = l.d.cout;
    a.kh = l.d.kh; a.kw = l.d.kw; a.stride = l.d.stride; a.pad = l.d.pad; a.groups = l.d.groups;
    a.act = l.d.act; a.pool = l.d.pool;
    if (net->ws) {
        a.splitk_ws = net->ws + net->splitk_off;
        a.splitk_bytes = kSplitKBytes;
    }
    return a;
}

static MbconvArgs mbconv_args(const dlf_net* net, int first, int last, const void* in_dev, void* out_dev) {
    MbconvArgs a;
    std::memset(&a, 0, sizeof(a));
    const Layer& f = net->layers[first];
    const Layer& z = net->layers[last];
    const bool has_expand = f.d.op == DLF_CONV;
    const Layer& dwl = net->layers[has_expand ? first + 1 : first];
    a.x = f.d.src < 0 ? in_dev : slot(net, f.d.src);
    a.w1 = has_expand ? f.w : nullptr; a.b1 = has_expand ? f.bias : nullptr;
    a.wd = dwl.w; a.bd = dwl.bias;
    a.w2 = z.w; a.b2 = z.bias;
    a.res = z.d.res_src == -2 ? nullptr : (z.d.res_src < 0 ? in_dev : slot(net, z.d.res_src));
    a.y = out_dev;
    a.N = static_cast<int>(f.in[0]); a.H = static_cast<int>(f.in[1]); a.W = static_cast<int>(f.in[2]);
    a.Cin = f.d.cin; a.hid = dwl.d.cin; a.Cout = z.d.cout; a.stride = dwl.d.stride;
    a.has_expand = has_expand ? 1 : 0;
    a.act1 = has_expand ? f.d.act : 0; a.act2 = dwl.d.act; a.act3 = z.d.act;
    return a;
}

// A fully connected layer is a 1x1 convolution over a 1x1 image whose channels are the flattened
// input (NHWC order, which is how the map lies in memory): the tensor-core kernel then streams the
// weight matrix through its TMA ring, one slab of output features per CTA.
static ConvArgs fc_as_conv_args(const dlf_net* net, int i, const void* in_dev, void* out_dev) {
    const Layer& l = net->layers[i];
    ConvArgs a;
    std::memset(&a, 0, sizeof(a));
    a.x = l.d.src < 0 ? in_dev : slot(net, l.d.src);
    a.w = l.w;
    a.bias = l.bias;
    a.y = out_dev;
    a.N = static_cast<int>(l.in[0]); a.H = 1; a.W = 1;
    a.Cin = l.d.cin; a.Ho = 1; a.Wo = 1; a.Cout = l.d.cout;
    a.kh = 1; a.kw = 1; a.stride = 1; a.pad = 0; a.groups = 1;
    a.act = l.d.act; a.pool = 0;
    if (net->ws) {
        a.splitk_ws = net->ws + net->splitk_off;
        a.splitk_bytes = kSplitKBytes;
    }
    return a;
}

// ---- projection branch + expansion layer of a residual block as ONE product -----------------------------------------------
// [1x1 projection (stride 1 or 2, linear) of the block's input, 1x1 expansion of the block's 3x3 output + that projection as
// residual]: y = act(x_e * W_e + b_e + x_p * W_p + b_p) is one implicit GEMM whose K runs over both inputs' channels, so the
// projection's map is never written nor read back; it joins the fp32 accumulator without its own fp16 rounding (at most half
// an fp16 unit in the last place of the projection's value away from the layer-by-layer result).
static bool span_is_projadd(const dlf_net* net, int first, int last) {
    if (net->opt_no_tc || last != first + 1) return false;
    const int n = static_cast<int>(net->layers.size());
    const dlf_layer_desc& pj = net->layers[first].d;
    const dlf_layer_desc& ex = net->layers[last].d;
    if (pj.op != DLF_CONV || ex.op != DLF_CONV || pj.groups != 1 || ex.groups != 1) return false;
    if (pj.kh != 1 || pj.kw != 1 || pj.pad != 0 || pj.pool || pj.res_src != -2 || pj.act != DLF_ACT_NONE) return false;
    if (ex.kh != 1 || ex.kw != 1 || ex.pad != 0 || ex.stride != 1 || ex.pool) return false;
    if (ex.res_src != first || ex.src == first || ex.src >= first) return false;
    for (int j = first + 1; j < n; j++) {   // the projection's map is used by the expansion layer's sum alone
        const dlf_layer_desc& d = net->layers[j].d;
        if (d.src == first || (d.res_src == first && j != last)) return false;
    }
    ConvArgs a = conv_args(net, last, nullptr, nullptr);
    a.res = nullptr;
    const Layer& pl = net->layers[first];
    a.x2 = &a;   // only whether there is one matters here
    a.H2 = static_cast<int>(pl.in[1]); a.W2 = static_cast<int>(pl.in[2]); a.Cin2 = pj.cin; a.stride2 = pj.stride;
    return conv_tc_dual_supported(a);
}

static ConvArgs projadd_args(const dlf_net* net, int first, int last, const void* in_dev, void* out_dev) {
    ConvArgs a = conv_args(net, last, in_dev, out_dev);
    const Layer& pl = net->layers[first];
    a.res = nullptr;
    a.splitk_ws = nullptr;
    a.splitk_bytes = 0;
    a.x2 = pl.d.src < 0 ? in_dev : slot(net, pl.d.src);
    a.w2 = pl.w;
    a.bias2 = pl.bias;
    a.H2 = static_cast<int>(pl.in[1]); a.W2 = static_cast<int>(pl.in[2]); a.Cin2 = pl.d.cin; a.stride2 = pl.d.stride;
    return a;
}

// ---- groups handed over through L2 -------------------------------------------------------------------------------------
// Any run of dense convolutions the single-layer tensor-core kernel takes (any kernel size, stride 1 or 2, fused pool,
// residual from anywhere, a projection branch) can run as ONE persistent kernel whose CTAs walk the layers together with a
// device-wide barrier in between; every layer's map goes to its workspace slot.
static bool span_is_seq(const dlf_net* net, int first, int last) {
    if (net->opt_no_tc || last - first + 1 > conv_seq_max_layers()) return false;
    for (int i = first; i <= last; i++) {
        const Layer& l = net->layers[i];
        if (l.d.op != DLF_CONV || l.d.groups != 1) return false;
        ConvArgs a = conv_args(net, i, nullptr, nullptr);
        if (!conv_seq_layer_supported(a)) return false;
    }
    return true;
}

static bool single_kind(const dlf_net* net, int i, Kind* kind) {
    const Layer& l = net->layers[i];
    switch (l.d.op) {
        case DLF_CONV: {
            ConvArgs a = conv_args(net, i, nullptr, nullptr);
            if (l.d.res_src == -2) a.res = nullptr; else a.res = &a;  // only whether there is one matters here
            if (!net->opt_no_tc && conv_tc_supported(a)) { *kind = K_CONV_TC; return true; }
            if (!net->opt_no_tc && stem_tc_supported(a)) { *kind = K_STEM_TC; return true; }
            if (l.d.groups > 1 && (l.d.cout / l.d.groups) % 16 != 0) return false;
            *kind = K_CONV_DIRECT;
            return true;
        }
        case DLF_DWCONV:
            if (l.d.kh != 3 || l.d.kw != 3 || l.d.cin % 8 || l.d.pool) return false;
            *kind = K_DW;
            return true;
        case DLF_FC:
            if (l.d.cin % 8) return false;
            // the CUDA-core kernel re-reads the weights once per 8 images and keeps few bytes in flight: measured
            // faster only for small matrices at small batch
            if (!net->opt_no_tc && l.d.res_src == -2 && (l.in[0] > 8 || l.w_elems * 2 >= (16ll << 20)) &&
                conv_tc_supported(fc_as_conv_args(net, i, nullptr, nullptr))) { *kind = K_CONV_TC; return true; }
            *kind = K_FC;
            return true;
        case DLF_MAXPOOL:
            if (l.d.cin % 8) return false;
            *kind = K_MAXPOOL;
            return true;
        case DLF_GAVGPOOL:
            if (l.d.cin % 8) return false;
            *kind = K_GAVG;
            return true;
    }
    return false;
}

static bool chain_pays(const dlf_net* net, int first, int last, int sms, ChainTiling* tiling);

static bool make_group(const dlf_net* net, int first, int last, int sms, Group* g) {
    g->first = first; g->last = last; g->sms = sms;
    g->tiling = ChainTiling{};
    g->mb_tiling = MbconvTiling{};
    if (first == last) {
        // A single layer runs through the single-layer kernels unless the option asks for the fused-group kernel
        // (a narrow 3x3 layer: 20.5 us in the single-layer kernel's row mode against 26 us here at 56x56x64, batch 32).
        // ... or the layer is a narrow 3x3 layer on an image too wide for the single-layer kernel's row mode (more than 126
        // pixels): that kernel then re-loads the input window for each of the nine taps, the fused-group kernel loads the
        // tile's frame once and shifts the operand window (VGG-16's 64 -> 64 layer at 224x224, batch 8: 74.5 -> 52.7 us).
        const Layer& l1 = net->layers[first];
        const bool wide_narrow = l1.d.op == DLF_CONV && l1.d.kh == 3 && l1.d.kw == 3 && l1.d.stride == 1 && l1.d.pad == 1 &&
                                 l1.d.cin <= 64 && l1.d.cout <= 64 && l1.wo_pre + 2 > 128;
        const bool prefer_chain = net->opt_single_chain != 0 || wide_narrow;
        if (!(prefer_chain && !net->opt_no_tc && span_is_chain(net, first, last))) return single_kind(net, first, &g->kind);
    }
    if (net->opt_no_tc) return false;
    if (first < last && span_is_mbconv(net, first, last, false)) {
        g->mb_tiling = mbconv_tiling(mbconv_args(net, first, last, nullptr, nullptr), sms);
        g->kind = K_MBCONV;
        return g->mb_tiling.ok;
    }
    if (span_is_projadd(net, first, last)) {
        g->kind = K_CONV_DUAL;
        return true;
    }
    // Two ways to fuse dense convolutions: hand-over in shared memory (a chain of stride-1 1x1 / 3x3 layers, tile by tile) or
    // through L2 (any run of dense convolutions, layer by layer behind a device-wide barrier).  Unless an option says
    // otherwise the first is taken for narrow layers (at most 64 channels: there it was measured faster), the second elsewhere.
    const bool chain_ok = span_is_chain(net, first, last);
    const bool seq_ok = first < last && span_is_seq(net, first, last);
    bool narrow = true;
    for (int i = first; i <= last; i++) narrow = narrow && net->layers[i].d.cin <= 64 && net->layers[i].d.cout <= 64;
    bool want_chain = chain_ok && (first == last || net->opt_group_kernel == 1 || (net->opt_group_kernel == 0 && narrow) || !seq_ok);
    if (chain_ok && !want_chain && net->opt_group_kernel == 0) {   // wide layers: where the estimate says the kernel pays (few tiles per SM)
        want_chain = chain_pays(net, first, last, sms, &g->tiling);
        if (want_chain) {
            g->kind = K_CHAIN_TC;
            return true;
        }
        g->tiling = ChainTiling{};
    }
    if (want_chain) {
        ChainArgs a = chain_args(net, first, last, nullptr, nullptr);
        g->tiling = chain_tc_tiling(a, sms, net->dev_sms);
        g->kind = K_CHAIN_TC;
        if (g->tiling.ok) return true;
        if (first == last) return single_kind(net, first, &g->kind);
    }
    if (seq_ok) {
        g->kind = K_CONV_SEQ;
        return true;
    }
    return false;
}

// ---- what the tuner may propose as one group --------------------------------------------------------------------
// Algorithm 1 grows a block while the layers can run as one kernel AND that kernel is expected to pay (Sec. IV-B: fusing
// helps layers with few operations and hurts heavy ones).  For a dense chain the estimate is the fused kernel's own cost
// model (the tiler's SM clocks at 1.9 GHz, plus one kernel boundary) against one kernel per layer: the slower of a layer's
// operations at 600 TFLOP/s and its bytes at 5.5 TB/s (what the single-layer kernel reaches on this chip) plus 7 us of
// fixed cost per kernel (measured: no single-layer kernel takes less inside a network); the group must win by 15 %
// (estimate and measurement differ by up to a quarter either way; groups that merely break even lose inside a network).
// A chain may not swallow the expansion layer of an inverted-residual block (the layer a depthwise convolution reads):
// that block fuses better as a whole.  Inverted-residual blocks follow the measured rule on the hidden width.  Groups
// handed over through L2 are proposed only when the option asks for them (measured: a device-wide barrier per layer is no
// cheaper than a kernel boundary).  `prefix`: the layers may also be the beginning of a pattern that can still grow.
// The estimate for a dense chain handed over in shared memory: true if the fused kernel is expected to beat one kernel per
// layer on `sms` SMs (see above).  `tiling` receives the fused kernel's tiling.
static bool chain_pays(const dlf_net* net, int first, int last, int sms, ChainTiling* tiling) {
    const ChainTiling t = chain_tc_tiling(chain_args(net, first, last, nullptr, nullptr), sms, net->dev_sms > 0 ? net->dev_sms : sms);
    if (tiling) *tiling = t;
    if (!t.ok) return false;
    double single_us = 0.0;
    for (int i = first; i <= last; i++) {
        const Layer& l = net->layers[i];
        const double bytes = static_cast<double>(l.in[0] * l.in[1] * l.in[2] * l.in[3] * 2) + static_cast<double>(l.bytes) + static_cast<double>(l.w_elems * 2) +
                             (l.d.res_src != -2 ? static_cast<double>(l.bytes) : 0.0);
        single_us += std::max(static_cast<double>(l.flops) / 600e6, bytes / 5.5e6) + 7.0;
    }
    return t.cost / 1.9e3 + 5.5 < 0.85 * single_us;
}

// The estimate for an inverted-residual block: the fused kernel's own cost model (the tiler's SM clocks, plus one kernel
// boundary) against one kernel per layer, each at its bytes at 2.5 TB/s - what the depthwise and the narrow pointwise kernels
// reach on this chip - plus 5 us of fixed cost; the block must win by a tenth.  It replaces the fixed limit on the hidden
// width of the first version: wide blocks on small maps (many 64-channel steps, few tiles to spread over the SMs) lose, the
// same blocks at a large batch win.
static bool mbconv_pays(const dlf_net* net, int first, int last, int sms) {
    const MbconvTiling t = mbconv_tiling(mbconv_args(net, first, last, nullptr, nullptr), sms);
    if (!t.ok) return false;
    double single_us = 0.0;
    for (int i = first; i <= last; i++) {
        const Layer& l = net->layers[i];
        const double bytes = static_cast<double>(l.in[0] * l.in[1] * l.in[2] * l.in[3] * 2) + static_cast<double>(l.bytes) + static_cast<double>(l.w_elems * 2) +
                             (l.d.res_src != -2 ? static_cast<double>(l.bytes) : 0.0);
        single_us += std::max(static_cast<double>(l.flops) / 600e6, bytes / 2.5e6) + 5.0;
    }
    return t.cost / 1.9e3 + 5.5 < 0.9 * single_us;
}

static bool tuner_may_fuse(const dlf_net* net, int first, int last, bool prefix, int s_max) {
    if (first == last) return true;
    if (net->opt_no_tc) return false;
    if (span_is_mbconv(net, first, last, prefix)) {
        // (the layers may be the beginning of the block: the estimate is made for the whole of it)
        const int full_last = first + (net->layers[first].d.op == DLF_CONV ? 2 : 1);
        return full_last < static_cast<int>(net->layers.size()) && span_is_mbconv(net, first, full_last, false) && mbconv_pays(net, first, full_last, s_max);
    }
    if (net->opt_group_kernel == 2 && span_is_seq(net, first, last)) return true;
    // a projection and the expansion layer it is added to are one product with a longer K: never slower than the two kernels
    if (span_is_projadd(net, first, last)) return true;
    if (!span_is_chain(net, first, last)) return false;
    if (net->opt_group_kernel == 1) return true;
    const int n = static_cast<int>(net->layers.size());
    for (int i = first; i <= last; i++)
        if (i + 1 < n && net->layers[i + 1].d.op == DLF_DWCONV && net->layers[i + 1].d.src == i) return false;
    return chain_pays(net, first, last, s_max, nullptr);
}

static int launch_group(dlf_net* net, const Group& g, const void* in_dev, void* final_out, cudaStream_t s) {
    const int n = static_cast<int>(net->layers.size());
    const Layer& z = net->layers[g.last];
    void* y = (g.last == n - 1) ? final_out : static_cast<void*>(net->ws + z.off);
    int* status = reinterpret_cast<int*>(net->ws + net->status_off);
    switch (g.kind) {
        case K_CHAIN_TC: {
            ChainArgs a = chain_args(net, g.first, g.last, in_dev, y);
            return launch_chain_tc(a, g.tiling, g.sms, status, s);
        }
        case K_CONV_SEQ: {
            ConvArgs a[16];
            const int cnt = g.last - g.first + 1;
            if (cnt > 16) return DLF_E_PLAN;
            for (int i = g.first; i <= g.last; i++)
                a[i - g.first] = conv_args(net, i, in_dev, i == n - 1 ? final_out : static_cast<void*>(net->ws + net->layers[i].off));
            return launch_conv_seq(a, cnt, g.sms, status, reinterpret_cast<unsigned*>(status) + 2, s);
        }
        case K_MBCONV: return launch_mbconv_tc(mbconv_args(net, g.first, g.last, in_dev, y), g.mb_tiling, g.sms, status, s);
        case K_CONV_TC:
            if (z.d.op == DLF_FC) return launch_conv_tc(fc_as_conv_args(net, g.first, in_dev, y), g.sms, status, s);
            return launch_conv_tc(conv_args(net, g.first, in_dev, y), g.sms, status, s);
        case K_CONV_DUAL: return launch_conv_tc(projadd_args(net, g.first, g.last, in_dev, y), g.sms, status, s);
        case K_STEM_TC: return launch_stem_tc(conv_args(net, g.first, in_dev, y), g.sms, status, s);
        case K_CONV_DIRECT: return launch_conv_direct(conv_args(net, g.first, in_dev, y), g.sms, s);
        case K_DW: return launch_dw3x3(conv_args(net, g.first, in_dev, y), g.sms, s);
        case K_FC: {
            const void* x = z.d.src < 0 ? in_dev : net->ws + net->layers[z.d.src].off;
            return launch_fc(x, z.w, z.bias, y, static_cast<int>(z.in[0]), z.d.cin, z.d.cout, z.d.act, g.sms, s);
        }
        case K_MAXPOOL: {
            const void* x = z.d.src < 0 ? in_dev : net->ws + net->layers[z.d.src].off;
            return launch_maxpool(x, y, static_cast<int>(z.in[0]), static_cast<int>(z.in[1]), static_cast<int>(z.in[2]),
                                  z.d.cin, z.d.kh, z.d.stride, z.d.pad, static_cast<int>(z.out[1]),
                                  static_cast<int>(z.out[2]), g.sms, s);
        }
        case K_GAVG: {
            const void* x = z.d.src < 0 ? in_dev : net->ws + net->layers[z.d.src].off;
            return launch_gavgpool(x, y, static_cast<int>(z.in[0]), static_cast<int>(z.in[1]), static_cast<int>(z.in[2]),
                                   z.d.cin, g.sms, s);
        }
    }
    return DLF_E_UNSUPPORTED;
}

}  // namespace dlf
namespace dlf {
int kernels_init() {
    int rc = conv_tc_init();
    if (rc == DLF_OK) rc = chain_tc_init();
    if (rc == DLF_OK) rc = mbconv_tc_init();
    return rc ? rc : stem_tc_init();
}

static void invalidate_graphs(dlf_net* net) {
    net->graph.drop();
    net->graph_timed.drop();
}

// Captures the launches of every group of the plan into one executable graph (thread-local
// capture on a stream the net owns, so that nothing else the caller's thread or other threads
// enqueue is swallowed).  With `timed`, an event is recorded before the first and after every group.
static int build_graph(dlf_net* net, GraphCache* gc, const void* in_dev, void* out_dev, bool timed) {
    gc->drop();
    cudaError_t e;
    if (!net->capture_stream) {
        e = cudaStreamCreateWithFlags(&net->capture_stream, cudaStreamNonBlocking);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (timed) {
        while (net->group_events.size() < net->plan.size() + 1) {
            cudaEvent_t ev;
            e = cudaEventCreate(&ev);
            if (e != cudaSuccess) return cuda_fail(e);
            net->group_events.push_back(ev);
        }
    }
    cudaStream_t cs = net->capture_stream;
    e = cudaStreamBeginCapture(cs, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) return cuda_fail(e);
    int rc = DLF_OK;
    if (timed) cudaEventRecordWithFlags(net->group_events[0], cs, cudaEventRecordExternal);
    for (size_t g = 0; g < net->plan.size() && rc == DLF_OK; g++) {
        rc = launch_group(net, net->plan[g], in_dev, out_dev, cs);
        if (timed && rc == DLF_OK) cudaEventRecordWithFlags(net->group_events[g + 1], cs, cudaEventRecordExternal);
    }
    cudaGraph_t graph = nullptr;
    e = cudaStreamEndCapture(cs, &graph);
    if (rc != DLF_OK) {
        if (graph) cudaGraphDestroy(graph);
        return rc;
    }
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaGraphInstantiate(&gc->exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) {
        gc->exec = nullptr;
        return cuda_fail(e);
    }
    gc->in = in_dev;
    gc->out = out_dev;
    return DLF_OK;
}

static int run_graph(dlf_net* net, GraphCache* gc, const void* in_dev, void* out_dev, bool timed, cudaStream_t s) {
    if (!gc->exec || gc->in != in_dev || gc->out != out_dev) {
        int rc = build_graph(net, gc, in_dev, out_dev, timed);
        if (rc) return rc;
    }
    cudaError_t e = cudaGraphLaunch(gc->exec, s);
    return e == cudaSuccess ? DLF_OK : cuda_fail(e);
}

static int check_ready(const dlf_net* net) {
    if (!net->ws) return DLF_E_WORKSPACE;
    if (net->plan.empty()) return DLF_E_STATE;
    for (const Layer& l : net->layers)
        if (is_param(l) && (!l.w || !l.bias)) return DLF_E_STATE;
    return DLF_OK;
}

static int validate_plan(const dlf_net* net, int n_groups, const int32_t* ends, const int32_t* sms, std::vector<Group>* out) {
    const int n = static_cast<int>(net->layers.size());
    if (n_groups < 1 || n_groups > n) return DLF_E_PLAN;
    std::vector<char> is_end(n, 0);
    int prev = -1;
    for (int g = 0; g < n_groups; g++) {
        if (ends[g] <= prev || ends[g] >= n) return DLF_E_PLAN;
        if (sms[g] < 1 || sms[g] > net->dev_sms) return DLF_E_PLAN;
        prev = ends[g];
        is_end[prev] = 1;
    }
    if (prev != n - 1) return DLF_E_PLAN;
    int first = 0;
    out->clear();
    std::vector<char> stored(n, 0);   // the layer's map reaches its workspace slot: a group's last layer, any layer of an L2 group
    for (int g = 0; g < n_groups; g++) {
        Group grp;
        if (!make_group(net, first, ends[g], sms[g], &grp)) return DLF_E_PLAN;
        out->push_back(grp);
        for (int i = first; i <= ends[g]; i++) stored[i] = (i == ends[g] || grp.kind == K_CONV_SEQ) ? 1 : 0;
        first = ends[g] + 1;
    }
    // a tensor read across a group boundary must have been stored
    first = 0;
    for (int g = 0; g < n_groups; g++) {
        for (int i = first; i <= ends[g]; i++) {
            const int refs[2] = {net->layers[i].d.src, net->layers[i].d.res_src};
            for (int r : refs)
                if (r >= 0 && r < first && !stored[r]) return DLF_E_PLAN;
        }
        first = ends[g] + 1;
    }
    return DLF_OK;
}

// Eq. 5 mapped to an SM count.
static int layer_sms(const Layer& l, const dlf_tuner_params& p, int s_max) {
    const double score = p.alpha * std::log2(static_cast<double>(l.d.cout)) + p.beta * std::log2(static_cast<double>(l.flops));
    const double s = std::floor(p.kappa * score + p.kappa0 + 0.5);
    return static_cast<int>(std::min<double>(std::max<double>(s, 1.0), s_max));
}

}  // namespace dlf

namespace dlf {
// The search's second half: given the best time t[a][len-1] of every span a..a+len-1 (infinity: cannot run) and the SM
// count that reached it, the contiguous partition with the least total time (a plan's time is the sum of its groups').
static int solve_partition(int n, int max_len, const std::vector<std::vector<float>>& t, const std::vector<std::vector<int>>& ts, int* n_groups,
                           int32_t* group_end, int32_t* sm_count, float* best_ms) {
    const float inf = std::numeric_limits<float>::infinity();
    std::vector<float> best(n + 1, inf);
    std::vector<int> from(n + 1, -1);
    best[0] = 0.0f;
    for (int i = 1; i <= n; i++)
        for (int len = 1; len <= max_len && len <= i; len++) {
            const int a = i - len;
            if (best[a] == inf || t[a][len - 1] == inf) continue;
            if (best[a] + t[a][len - 1] < best[i]) { best[i] = best[a] + t[a][len - 1]; from[i] = a; }
        }
    if (best[n] == inf) return DLF_E_PLAN;
    std::vector<int> cuts;
    for (int i = n; i > 0; i = from[i]) cuts.push_back(i);
    std::reverse(cuts.begin(), cuts.end());
    int a = 0;
    for (size_t g = 0; g < cuts.size(); g++) {
        group_end[g] = cuts[g] - 1;
        sm_count[g] = ts[a][cuts[g] - a - 1];
        a = cuts[g];
    }
    *n_groups = static_cast<int>(cuts.size());
    if (best_ms) *best_ms = best[n];
    return DLF_OK;
}
}  // namespace dlf

dlf_net::~dlf_net() {
    graph.drop();
    graph_timed.drop();
    for (cudaEvent_t ev : group_events) cudaEventDestroy(ev);
    if (capture_stream) cudaStreamDestroy(capture_stream);
}

// ---- C ABI ------------------------------------------------------------------------------------------

extern "C" {

const char* dlf_strerror(int status) {
    switch (status) {
        case DLF_OK: return "ok";
        case DLF_E_INVALID_ARG: return "invalid argument";
        case DLF_E_SHAPE: return "layer list does not type-check";
        case DLF_E_PLAN: return "invalid fusion plan";
        case DLF_E_WORKSPACE: return "workspace missing, misaligned or too small";
        case DLF_E_UNSUPPORTED: return "unsupported layer";
        case DLF_E_CUDA: return "CUDA error";
        case DLF_E_TIMEOUT: return "device-side wait timed out";
        case DLF_E_STATE: return "call out of order (weights, plan or workspace missing)";
    }
    return "unknown status";
}

int dlf_last_cuda_error(void) { return g_last_cuda_error; }

int dlf_device_sm_count(void) {
    int sms = 0;
    int rc = query_sms(&sms);
    return rc ? rc : sms;
}

int dlf_net_create(const dlf_layer_desc* layers, int n_layers, int N, int H, int W, int C, dlf_net** out) {
    if (!layers || !out || n_layers <= 0 || N <= 0 || H <= 0 || W <= 0 || C <= 0) return DLF_E_INVALID_ARG;
    *out = nullptr;
    dlf_net* net = new (std::nothrow) dlf_net();
    if (!net) return DLF_E_INVALID_ARG;
    net->N = N; net->H = H; net->W = W; net->C = C;
    net->layers.resize(n_layers);
    int rc = DLF_OK;
    size_t off = 0;
    net->in_off = 0;
    net->in_bytes = static_cast<size_t>(N) * H * W * C * 2;
    off = align_up(net->in_bytes, 256);
    for (int i = 0; i < n_layers && rc == DLF_OK; i++) {
        Layer& l = net->layers[i];
        l.d = layers[i];
        l.w = nullptr; l.bias = nullptr;
        const dlf_layer_desc& d = l.d;
        if (d.op < DLF_CONV || d.op > DLF_GAVGPOOL || d.act < DLF_ACT_NONE || d.act > DLF_ACT_RELU6) { rc = DLF_E_INVALID_ARG; break; }
        if (d.src < -1 || d.src >= i || d.res_src < -2 || d.res_src >= i) { rc = DLF_E_SHAPE; break; }
        const int64_t* in = nullptr;
        int64_t net_in[4] = {N, H, W, C};
        in = d.src < 0 ? net_in : net->layers[d.src].out;
        std::memcpy(l.in, in, sizeof(l.in));
        l.ops_eq1 = l.flops = l.w_elems = 0;
        if (d.op == DLF_CONV || d.op == DLF_DWCONV || d.op == DLF_MAXPOOL) {
            if (d.kh <= 0 || d.kw <= 0 || d.stride <= 0 || d.pad < 0) { rc = DLF_E_INVALID_ARG; break; }
            if (d.cin != in[3]) { rc = DLF_E_SHAPE; break; }
            const int64_t ho = (in[1] + 2 * d.pad - d.kh) / d.stride + 1, wo = (in[2] + 2 * d.pad - d.kw) / d.stride + 1;
            if (in[1] + 2 * d.pad < d.kh || in[2] + 2 * d.pad < d.kw || ho <= 0 || wo <= 0) { rc = DLF_E_SHAPE; break; }
            l.ho_pre = static_cast<int>(ho); l.wo_pre = static_cast<int>(wo);
            if (d.op == DLF_MAXPOOL) {
                if (d.cout != d.cin || d.pad >= d.kh || d.pool != 0 || d.res_src != -2) { rc = DLF_E_SHAPE; break; }
                l.out[0] = in[0]; l.out[1] = ho; l.out[2] = wo; l.out[3] = d.cin;
            } else {
                if (d.groups <= 0 || d.cin % d.groups || d.cout % d.groups || d.cout <= 0) { rc = DLF_E_SHAPE; break; }
                if (d.op == DLF_DWCONV && !(d.groups == d.cin && d.cin == d.cout)) { rc = DLF_E_SHAPE; break; }
                if (d.pool != 0 && d.pool != 2) { rc = DLF_E_INVALID_ARG; break; }
                const int64_t hp = d.pool ? ho / 2 : ho, wp = d.pool ? wo / 2 : wo;
                if (hp <= 0 || wp <= 0) { rc = DLF_E_SHAPE; break; }
                l.out[0] = in[0]; l.out[1] = hp; l.out[2] = wp; l.out[3] = d.cout;
                l.ops_eq1 = 2 * ho * wo * d.kh * d.kw * static_cast<int64_t>(d.cin) * d.cout;
                l.flops = l.ops_eq1 * in[0] / d.groups;
                l.w_elems = static_cast<int64_t>(d.cout) * d.kh * d.kw * (d.cin / d.groups);
            }
        } else if (d.op == DLF_FC) {
            if (d.cin != in[1] * in[2] * in[3] || d.cout <= 0 || d.pool != 0) { rc = DLF_E_SHAPE; break; }
            l.out[0] = in[0]; l.out[1] = 1; l.out[2] = 1; l.out[3] = d.cout;
            l.ops_eq1 = 2 * static_cast<int64_t>(d.cin) * d.cout;
            l.flops = l.ops_eq1 * in[0];
            l.w_elems = static_cast<int64_t>(d.cin) * d.cout;
            l.ho_pre = l.wo_pre = 1;
        } else {  // global average pool
            if (d.cin != in[3] || d.cout != d.cin || d.pool != 0 || d.res_src != -2) { rc = DLF_E_SHAPE; break; }
            l.out[0] = in[0]; l.out[1] = 1; l.out[2] = 1; l.out[3] = d.cin;
            l.ho_pre = l.wo_pre = 1;
        }
        if (d.res_src != -2) {
            // the residual must have the shape of the pre-pool output
            int64_t rs[4];
            std::memcpy(rs, d.res_src < 0 ? net_in : net->layers[d.res_src].out, sizeof(rs));
            if (rs[0] != l.out[0] || rs[1] != l.ho_pre || rs[2] != l.wo_pre || rs[3] != l.out[3]) { rc = DLF_E_SHAPE; break; }
        }
        l.bytes = static_cast<size_t>(l.out[0] * l.out[1] * l.out[2] * l.out[3]) * 2;
        l.off = off;
        off = align_up(off + l.bytes, 256);
    }
    if (rc == DLF_OK) {
        // every layer must have a kernel
        for (int i = 0; i < n_layers; i++) {
            Kind k;
            if (!single_kind(net, i, &k)) { rc = DLF_E_UNSUPPORTED; break; }
        }
    }
    if (rc != DLF_OK) {
        delete net;
        return rc;
    }
    net->status_off = off;
    net->splitk_off = off + 256;
    net->ws_need = net->splitk_off + kSplitKBytes;
    *out = net;
    return DLF_OK;
}

void dlf_net_destroy(dlf_net* net) { delete net; }

int dlf_net_layer_info(const dlf_net* net, int layer, int64_t* ops_eq1, int64_t* flops, int64_t out_shape[4]) {
    if (!net || layer < 0 || layer >= static_cast<int>(net->layers.size())) return DLF_E_INVALID_ARG;
    const Layer& l = net->layers[layer];
    if (ops_eq1) *ops_eq1 = l.ops_eq1;
    if (flops) *flops = l.flops;
    if (out_shape) std::memcpy(out_shape, l.out, sizeof(l.out));
    return DLF_OK;
}

int dlf_net_set_weights(dlf_net* net, int layer, const void* w_f16_dev, const float* bias_dev) {
    if (!net || layer < 0 || layer >= static_cast<int>(net->layers.size()) || !w_f16_dev || !bias_dev) return DLF_E_INVALID_ARG;
    Layer& l = net->layers[layer];
    if (!is_param(l)) return DLF_E_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(w_f16_dev) & 15) || (reinterpret_cast<uintptr_t>(bias_dev) & 15)) return DLF_E_INVALID_ARG;
    l.w = w_f16_dev;
    invalidate_graphs(net);
    l.bias = bias_dev;
    return DLF_OK;
}

int dlf_net_workspace_bytes(const dlf_net* net, size_t* bytes) {
    if (!net || !bytes) return DLF_E_INVALID_ARG;
    *bytes = net->ws_need;
    return DLF_OK;
}

int dlf_net_bind_workspace(dlf_net* net, void* workspace_dev, size_t bytes) {
    if (!net) return DLF_E_INVALID_ARG;
    if (!workspace_dev || (reinterpret_cast<uintptr_t>(workspace_dev) & 255) || bytes < net->ws_need) return DLF_E_WORKSPACE;
    if (net->dev_sms == 0) {
        int rc = query_sms(&net->dev_sms);
        if (rc) return rc;
    }
    net->ws = static_cast<uint8_t*>(workspace_dev);
    invalidate_graphs(net);
    net->ws_bytes = bytes;
    // the status block and, behind it, the split-K arrival counters (zero between launches)
    cudaError_t e = cudaMemset(net->ws + net->status_off, 0, 256 + kSplitKCounterBytes);
    if (e != cudaSuccess) return cuda_fail(e);
    return DLF_OK;
}

int dlf_net_set_plan(dlf_net* net, int n_groups, const int32_t* group_end, const int32_t* sm_count) {
    if (!net || !group_end || !sm_count) return DLF_E_INVALID_ARG;
    if (net->dev_sms == 0) {
        int rc = query_sms(&net->dev_sms);
        if (rc) return rc;
    }
    std::vector<Group> plan;
    int rc = validate_plan(net, n_groups, group_end, sm_count, &plan);
    if (rc) return rc;
    rc = kernels_init();
    if (rc) return rc;
    net->plan.swap(plan);
    invalidate_graphs(net);
    return DLF_OK;
}

int dlf_net_plan_unfused(dlf_net* net) {
    if (!net) return DLF_E_INVALID_ARG;
    if (net->dev_sms == 0) {
        int rc = query_sms(&net->dev_sms);
        if (rc) return rc;
    }
    const int n = static_cast<int>(net->layers.size());
    std::vector<int32_t> ends(n), sms(n, net->dev_sms);
    for (int i = 0; i < n; i++) ends[i] = i;
    return dlf_net_set_plan(net, n, ends.data(), sms.data());
}

int dlf_net_get_plan(const dlf_net* net, int* n_groups, int32_t* group_end, int32_t* sm_count) {
    if (!net || !n_groups || !group_end || !sm_count) return DLF_E_INVALID_ARG;
    *n_groups = static_cast<int>(net->plan.size());
    for (size_t g = 0; g < net->plan.size(); g++) {
        group_end[g] = net->plan[g].last;
        sm_count[g] = net->plan[g].sms;
    }
    return DLF_OK;
}

int dlf_net_group_is_legal(const dlf_net* net, int first, int last, int sm_count) {
    if (!net || first < 0 || last < first || last >= static_cast<int>(net->layers.size())) return DLF_E_INVALID_ARG;
    if (net->dev_sms == 0) {
        int rc = query_sms(&const_cast<dlf_net*>(net)->dev_sms);
        if (rc) return rc;
    }
    if (sm_count < 1 || sm_count > net->dev_sms) return 0;
    Group g;
    return make_group(net, first, last, sm_count, &g) ? 1 : 0;
}

int dlf_net_tuner_may_fuse(const dlf_net* net, int first, int last, int prefix, int s_max) {
    if (!net || first < 0 || last < first || last >= static_cast<int>(net->layers.size()) || s_max < 1) return DLF_E_INVALID_ARG;
    return tuner_may_fuse(net, first, last, prefix != 0, s_max) ? 1 : 0;
}

int dlf_net_autotune(const dlf_net* net, const dlf_tuner_params* params, int* n_groups, int32_t* group_end,
                     int32_t* sm_count) {
    if (!net || !params || !n_groups || !group_end || !sm_count) return DLF_E_INVALID_ARG;
    int s_max = params->s_max;
    if (s_max <= 0 || params->legalise) {
        int sms = net->dev_sms;
        if (sms == 0) {
            int rc = query_sms(&sms);
            if (rc) return rc;
            const_cast<dlf_net*>(net)->dev_sms = sms;
        }
        if (s_max <= 0 || s_max > sms) s_max = sms;
    }
    if (!(params->op_critical > 0.0)) return DLF_E_INVALID_ARG;
    const int n = static_cast<int>(net->layers.size());
    double sum_op = 0.0, sum_mp = 0.0;
    int block = 0, start = 0, ng = 0;
    for (int i = 0; i < n; i++) {
        const Layer& l = net->layers[i];
        if (is_param(l)) {
            sum_op += static_cast<double>(l.flops);
            sum_mp += layer_sms(l, *params, s_max);
            block++;
        }
        // a block may grow while its layers are, or can still become, a group one kernel runs; it may
        // close only where they already are one (inside an inverted-residual block it keeps growing)
        bool forced = (i == n - 1) || !tuner_may_fuse(net, start, i + 1, true, s_max);
        const bool closable = (i == start) || tuner_may_fuse(net, start, i, false, s_max);
        if (!forced && params->legalise) {
            Group g;
            if (i + 1 > start && tuner_may_fuse(net, start, i + 1, false, s_max))
                forced = !make_group(net, start, i + 1, s_max, &g);
        }
        if (block > 0) {
            const double avg = sum_mp / block;
            if ((sum_op / avg >= params->op_critical && closable) || forced) {
                int mp = 1 << static_cast<int>(std::floor(std::log2(avg)));
                if (avg >= s_max) mp = s_max;  // the top step is the whole chip, as 32 of 32 cores in the paper
                mp = std::min(std::max(mp, 1), s_max);
                Group g;
                if (params->legalise && i > start && !make_group(net, start, i, mp, &g)) {
                    // the block cannot run as one kernel: one group per layer
                    for (int j = start; j <= i; j++) { group_end[ng] = j; sm_count[ng] = mp; ng++; }
                } else {
                    group_end[ng] = i;
                    sm_count[ng] = mp;
                    ng++;
                }
                sum_op = sum_mp = 0.0;
                block = 0;
                start = i + 1;
            }
        } else if (forced) {
            group_end[ng] = i;
            sm_count[ng] = s_max;
            ng++;
            start = i + 1;
        }
    }
    *n_groups = ng;
    return DLF_OK;
}

int dlf_net_run(dlf_net* net, const void* in_f16_dev, void* out_f16_dev, void* stream) {
    if (!net || !in_f16_dev || !out_f16_dev) return DLF_E_INVALID_ARG;
    int rc = check_ready(net);
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (net->opt_graph) {
        rc = run_graph(net, &net->graph, in_f16_dev, out_f16_dev, false, s);
        if (rc) return rc;
    } else {
        for (const Group& g : net->plan) {
            rc = launch_group(net, g, in_f16_dev, out_f16_dev, s);
            if (rc) return rc;
        }
    }
    net->last_out = out_f16_dev;
    return DLF_OK;
}

int dlf_net_sync(dlf_net* net, void* stream) {
    if (!net) return DLF_E_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    if (net->ws) {
        int st = 0;
        e = cudaMemcpy(&st, net->ws + net->status_off, sizeof(int), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return cuda_fail(e);
        if (st != 0) {
            g_last_cuda_error = st;
            cudaMemset(net->ws + net->status_off, 0, 4 * sizeof(int));   // the status word and the multi-layer kernels' barrier counters
            // a launch that gave up may have left split-K arrival counters behind
            cudaMemset(net->ws + net->splitk_off, 0, kSplitKCounterBytes);
            return DLF_E_TIMEOUT;
        }
    }
    return DLF_OK;
}

int dlf_net_debug_stall(dlf_net* net, int limit_us, void* stream) {
    if (!net || limit_us < 1 || limit_us > 1000000) return DLF_E_INVALID_ARG;
    if (!net->ws) return DLF_E_WORKSPACE;
    return launch_stall(reinterpret_cast<int*>(net->ws + net->status_off), static_cast<unsigned long long>(limit_us) * 1000ull,
                        static_cast<cudaStream_t>(stream));
}

int dlf_net_run_host(dlf_net* net, const void* in_f16_host, void* out_f16_host, void* stream) {
    if (!net || !in_f16_host || !out_f16_host) return DLF_E_INVALID_ARG;
    int rc = check_ready(net);
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const Layer& z = net->layers.back();
    cudaError_t e = cudaMemcpyAsync(net->ws + net->in_off, in_f16_host, net->in_bytes, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(e);
    rc = dlf_net_run(net, net->ws + net->in_off, net->ws + z.off, s);
    if (rc) return rc;
    e = cudaMemcpyAsync(out_f16_host, net->ws + z.off, z.bytes, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(e);
    return dlf_net_sync(net, s);
}

static float median_of(std::vector<float> v) {
    std::sort(v.begin(), v.end());
    return v.empty() ? 0.0f : v[v.size() / 2];
}

int dlf_net_time(dlf_net* net, const void* in_dev, void* out_dev, void* stream, int warmup, int iters, void* flush_dev,
                 size_t flush_bytes, float* ms_median, float* ms_min, float* ms_per_group) {
    if (!net || !in_dev || !out_dev || warmup < 0 || iters < 1) return DLF_E_INVALID_ARG;
    int rc = check_ready(net);
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t ng = net->plan.size();
    std::vector<cudaEvent_t> ev(2);
    for (auto& e : ev)
        if (cudaEventCreate(&e) != cudaSuccess) return cuda_fail(cudaGetLastError());
    auto cleanup = [&]() { for (auto& e : ev) cudaEventDestroy(e); };
    for (int i = 0; i < warmup; i++) {
        rc = dlf_net_run(net, in_dev, out_dev, s);
        if (rc) { cleanup(); return rc; }
    }
    std::vector<float> times;
    for (int i = 0; i < iters; i++) {
        if (flush_dev && flush_bytes) cudaMemsetAsync(flush_dev, i & 0xff, flush_bytes, s);
        cudaEventRecord(ev[0], s);
        rc = dlf_net_run(net, in_dev, out_dev, s);
        if (rc) { cleanup(); return rc; }
        cudaEventRecord(ev[1], s);
        cudaError_t e = cudaEventSynchronize(ev[1]);
        if (e != cudaSuccess) { cleanup(); return cuda_fail(e); }
        float ms = 0.0f;
        cudaEventElapsedTime(&ms, ev[0], ev[1]);
        times.push_back(ms);
    }
    if (ms_median) *ms_median = median_of(times);
    if (ms_min) *ms_min = *std::min_element(times.begin(), times.end());
    if (ms_per_group) {
        std::vector<std::vector<float>> per(ng);
        const int reps = std::min(std::max(iters, 3), 20);
        for (int i = 0; i < reps; i++) {
            if (flush_dev && flush_bytes) cudaMemsetAsync(flush_dev, i & 0xff, flush_bytes, s);
            rc = run_graph(net, &net->graph_timed, in_dev, out_dev, true, s);
            if (rc) { cleanup(); return rc; }
            cudaError_t e = cudaStreamSynchronize(s);
            if (e != cudaSuccess) { cleanup(); return cuda_fail(e); }
            for (size_t g = 0; g < ng; g++) {
                float ms = 0.0f;
                cudaEventElapsedTime(&ms, net->group_events[g], net->group_events[g + 1]);
                per[g].push_back(ms);
            }
        }
        for (size_t g = 0; g < ng; g++) ms_per_group[g] = median_of(per[g]);
    }
    cleanup();
    return dlf_net_sync(net, s);
}

// Median device time of ONE launch of group `g`: a graph of kReps back-to-back launches (which hides the
// host's launch cost) is timed `iters` times between two events after `warmup` untimed launches.
static int time_group(dlf_net* net, const Group& g, const void* in_dev, void* final_out, cudaStream_t s, cudaEvent_t e0,
                      cudaEvent_t e1, int warmup, int iters, float* ms_out) {
    const int kReps = 4;
    int rc = DLF_OK;
    cudaGraphExec_t exec = nullptr;
    if (!net->capture_stream && cudaStreamCreateWithFlags(&net->capture_stream, cudaStreamNonBlocking) != cudaSuccess)
        return cuda_fail(cudaGetLastError());
    cudaGraph_t graph = nullptr;
    if (cudaStreamBeginCapture(net->capture_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return cuda_fail(cudaGetLastError());
    for (int r = 0; r < kReps && rc == DLF_OK; r++) rc = launch_group(net, g, in_dev, final_out, net->capture_stream);
    cudaError_t e = cudaStreamEndCapture(net->capture_stream, &graph);
    if (rc == DLF_OK && e != cudaSuccess) rc = cuda_fail(e);
    if (rc == DLF_OK && cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) rc = cuda_fail(cudaGetLastError());
    if (graph) cudaGraphDestroy(graph);
    for (int i = 0; i < warmup && rc == DLF_OK; i++)
        if (cudaGraphLaunch(exec, s) != cudaSuccess) rc = cuda_fail(cudaGetLastError());
    std::vector<float> v;
    for (int i = 0; i < iters && rc == DLF_OK; i++) {
        cudaEventRecord(e0, s);
        if (cudaGraphLaunch(exec, s) != cudaSuccess) rc = cuda_fail(cudaGetLastError());
        cudaEventRecord(e1, s);
        if (rc == DLF_OK && cudaEventSynchronize(e1) != cudaSuccess) rc = cuda_fail(cudaGetLastError());
        float ms = 0.0f;
        if (rc == DLF_OK) cudaEventElapsedTime(&ms, e0, e1);
        v.push_back(ms / kReps);
    }
    if (exec) cudaGraphExecDestroy(exec);
    if (rc == DLF_OK) *ms_out = median_of(v);
    return rc;
}

int dlf_net_time_span(dlf_net* net, int first, int last, int sm_count, const void* in_dev, void* stream, int warmup,
                      int iters, int prepare, float* ms) {
    if (!net || !in_dev || !ms || first < 0 || last < first || last >= static_cast<int>(net->layers.size()) || warmup < 0 || iters < 1)
        return DLF_E_INVALID_ARG;
    if (!net->ws) return DLF_E_WORKSPACE;
    for (const Layer& l : net->layers)
        if (is_param(l) && (!l.w || !l.bias)) return DLF_E_STATE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    void* final_out = net->ws + net->layers.back().off;
    int rc = DLF_OK;
    if (prepare) {   // every layer's slot filled once, so that the span finds its inputs in HBM
        std::vector<Group> saved = net->plan;
        rc = dlf_net_plan_unfused(net);
        if (rc == DLF_OK) rc = dlf_net_run(net, in_dev, final_out, s);
        if (rc == DLF_OK) rc = dlf_net_sync(net, s);
        net->plan = saved;
        invalidate_graphs(net);
        if (rc) return rc;
    }
    if (net->dev_sms == 0) {
        rc = query_sms(&net->dev_sms);
        if (rc) return rc;
    }
    if (sm_count < 1 || sm_count > net->dev_sms) return DLF_E_PLAN;
    Group g;
    if (!make_group(net, first, last, sm_count, &g)) return DLF_E_PLAN;
    rc = kernels_init();
    if (rc) return rc;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return cuda_fail(cudaGetLastError());
    rc = time_group(net, g, in_dev, final_out, s, e0, e1, warmup, iters, ms);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return rc ? rc : dlf_net_sync(net, s);
}

int dlf_net_bruteforce(dlf_net* net, const dlf_search_params* sp, const void* in_dev, void* stream, int* n_groups,
                       int32_t* group_end, int32_t* sm_count, float* best_ms) {
    if (!net || !sp || !in_dev || !n_groups || !group_end || !sm_count) return DLF_E_INVALID_ARG;
    if (sp->n_sm_choices < 1 || sp->n_sm_choices > 16 || sp->max_group_len < 1 || sp->iters < 1 || sp->warmup < 0) return DLF_E_INVALID_ARG;
    if (!net->ws) return DLF_E_WORKSPACE;
    for (const Layer& l : net->layers)
        if (is_param(l) && (!l.w || !l.bias)) return DLF_E_STATE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int n = static_cast<int>(net->layers.size());
    std::vector<Group> saved = net->plan;
    // fill every layer's slot once so that each candidate group finds its inputs in HBM
    int rc = dlf_net_plan_unfused(net);
    if (rc) { net->plan = saved; invalidate_graphs(net); return rc; }
    void* final_out = net->ws + net->layers.back().off;
    rc = dlf_net_run(net, in_dev, final_out, s);
    if (rc == DLF_OK) rc = dlf_net_sync(net, s);
    net->plan = saved;
    invalidate_graphs(net);   // the graph just built holds the no-fusion plan
    if (rc) return rc;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return cuda_fail(cudaGetLastError());
    const float inf = std::numeric_limits<float>::infinity();
    // t[a][len-1] = best time of span a..a+len-1 over the SM choices
    std::vector<std::vector<float>> t(n, std::vector<float>(sp->max_group_len, inf));
    std::vector<std::vector<int>> ts(n, std::vector<int>(sp->max_group_len, 0));
    for (int a = 0; a < n && rc == DLF_OK; a++)
        for (int len = 1; len <= sp->max_group_len && a + len <= n && rc == DLF_OK; len++)
            for (int c = 0; c < sp->n_sm_choices && rc == DLF_OK; c++) {
                const int S = sp->sm_choices[c];
                if (S < 1 || S > net->dev_sms) continue;
                Group g;
                if (!make_group(net, a, a + len - 1, S, &g)) continue;
                float m = 0.0f;
                rc = time_group(net, g, in_dev, final_out, s, e0, e1, sp->warmup, sp->iters, &m);
                if (rc == DLF_OK && m < t[a][len - 1]) { t[a][len - 1] = m; ts[a][len - 1] = S; }
            }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc) return rc;
    rc = solve_partition(n, sp->max_group_len, t, ts, n_groups, group_end, sm_count, best_ms);
    if (rc) return rc;
    return dlf_net_sync(net, s);
}

int dlf_bruteforce_table(int n_layers, int max_group_len, int n_sm_choices, const int32_t* sm_choices, const float* ms, int* n_groups,
                         int32_t* group_end, int32_t* sm_count, float* best_ms) {
    if (n_layers < 1 || max_group_len < 1 || n_sm_choices < 1 || !sm_choices || !ms || !n_groups || !group_end || !sm_count) return DLF_E_INVALID_ARG;
    const float inf = std::numeric_limits<float>::infinity();
    std::vector<std::vector<float>> t(n_layers, std::vector<float>(max_group_len, inf));
    std::vector<std::vector<int>> ts(n_layers, std::vector<int>(max_group_len, 0));
    for (int a = 0; a < n_layers; a++)
        for (int len = 1; len <= max_group_len && a + len <= n_layers; len++)
            for (int c = 0; c < n_sm_choices; c++) {
                const float m = ms[(static_cast<size_t>(a) * max_group_len + (len - 1)) * n_sm_choices + c];
                if (m >= 0.0f && m < t[a][len - 1]) { t[a][len - 1] = m; ts[a][len - 1] = sm_choices[c]; }
            }
    return solve_partition(n_layers, max_group_len, t, ts, n_groups, group_end, sm_count, best_ms);

}

int dlf_net_boundary_tensor(const dlf_net* net, int layer, const void** dev_ptr, int64_t shape[4]) {
    if (!net || !dev_ptr || layer < 0 || layer >= static_cast<int>(net->layers.size())) return DLF_E_INVALID_ARG;
    if (!net->ws) return DLF_E_WORKSPACE;
    bool is_end = false;
    for (const Group& g : net->plan) is_end |= (g.last == layer);
    if (!is_end) return DLF_E_PLAN;
    const Layer& l = net->layers[layer];
    *dev_ptr = (layer == static_cast<int>(net->layers.size()) - 1) ? net->last_out : net->ws + l.off;
    if (shape) std::memcpy(shape, l.out, sizeof(l.out));
    return DLF_OK;
}

int dlf_net_group_model(const dlf_net* net, int group, int64_t* flops, int64_t* hbm_bytes, double* redundancy, int* launches) {
    if (!net || group < 0 || group >= static_cast<int>(net->plan.size())) return DLF_E_INVALID_ARG;
    const Group& g = net->plan[group];
    int64_t fl = 0, by = 0;
    const Layer& f = net->layers[g.first];
    const Layer& z = net->layers[g.last];
    by += f.in[0] * f.in[1] * f.in[2] * f.in[3] * 2;
    by += static_cast<int64_t>(z.bytes);
    for (int i = g.first; i <= g.last; i++) {
        const Layer& l = net->layers[i];
        fl += l.flops;
        by += l.w_elems * 2 + (is_param(l) ? l.d.cout * 4 : 0);
        if (l.d.res_src != -2 && l.d.res_src < g.first) by += l.out[0] * l.ho_pre * l.wo_pre * l.out[3] * 2;
        if (g.kind == K_CONV_DUAL && i > g.first) by += l.in[0] * l.in[1] * l.in[2] * l.in[3] * 2;   // the expansion layer's own input
        // a group handed over through L2 still writes every map to its slot and reads it back: counted like separate layers
        if (g.kind == K_CONV_SEQ) {
            if (i > g.first) by += l.in[0] * l.in[1] * l.in[2] * l.in[3] * 2;
            if (i < g.last) by += static_cast<int64_t>(l.bytes);
            if (l.d.res_src != -2 && l.d.res_src >= g.first) by += l.out[0] * l.ho_pre * l.wo_pre * l.out[3] * 2;
        }
    }
    if (flops) *flops = fl;
    if (hbm_bytes) *hbm_bytes = by;
    if (redundancy) *redundancy = g.kind == K_CHAIN_TC ? g.tiling.redundancy : (g.kind == K_MBCONV ? g.mb_tiling.redundancy : 1.0);
    if (launches) *launches = 1;
    return DLF_OK;
}

const char* dlf_net_group_kernel(const dlf_net* net, int group) {
    if (!net || group < 0 || group >= static_cast<int>(net->plan.size())) return "";
    return kKindName[net->plan[group].kind];
}

int dlf_net_set_option(dlf_net* net, int option, int value) {
    if (!net) return DLF_E_INVALID_ARG;
    switch (option) {
        case DLF_OPT_NO_TENSOR_CORE: net->opt_no_tc = value != 0; break;
        case DLF_OPT_SINGLE_AS_CHAIN: net->opt_single_chain = value != 0; break;
        case DLF_OPT_GROUP_KERNEL:
            if (value < 0 || value > 2) return DLF_E_INVALID_ARG;
            net->opt_group_kernel = value;
            break;
        case DLF_OPT_CUDA_GRAPH: net->opt_graph = value != 0; return DLF_OK;
        case DLF_OPT_PDL: g_use_pdl = value != 0; invalidate_graphs(net); return DLF_OK;
        case DLF_OPT_CONV_ROW_MODE:
            if (value < 0 || value > 2) return DLF_E_INVALID_ARG;
            g_conv_row_mode = value;
            invalidate_graphs(net);
            return DLF_OK;
        default: return DLF_E_INVALID_ARG;
    }
    net->plan.clear();  // kernel choices depend on the options: the plan must be set again
    invalidate_graphs(net);
    return DLF_OK;
}

}  // extern "C"
