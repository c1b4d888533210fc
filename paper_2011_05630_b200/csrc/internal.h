// Internal declarations shared by the host model, the launcher and the kernels' host wrappers.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/dlfusion.h"

namespace dlf {

// One convolution-like layer as a kernel sees it.  Ho, Wo are the sizes BEFORE a fused pool.
struct ConvArgs {
    const void* x;
    const void* w;
    const float* bias;
    const void* res;  // nullable, shape [N][Ho][Wo][Cout]
    void* y;          // [N][Ho][Wo][Cout], or [N][Ho/2][Wo/2][Cout] with pool == 2
    int N, H, W, Cin, Ho, Wo, Cout;
    int kh, kw, stride, pad, groups, act, pool;
    // Optional device scratch for split-K (fully connected layers at small batch): 64 KB of arrival counters that
    // are zero between launches, then room for fp32 partial tiles.  Null: every tile is one work item.
    void* splitk_ws;
    size_t splitk_bytes;
    // Optional second 1x1 source whose product joins the same accumulator (a residual block's projection branch fused
    // with its expansion layer): y = act(x * w + bias + x2 * w2 + bias2).  x2 is [N][H2][W2][Cin2], read at
    // (ho * stride2, wo * stride2); w2 is [Cout][Cin2].  Null x2: an ordinary layer.
    const void* x2;
    const void* w2;
    const float* bias2;
    int H2, W2, Cin2, stride2;
};

// True if `a` (with its second source) can run as one conv_tc launch.
bool conv_tc_dual_supported(const ConvArgs& a);

// A chain of stride-1, size-keeping dense convolutions executed by one kernel.
constexpr int kMaxChain = 8;
struct ChainArgs {
    int n_layers;
    const void* x;
    const void* w[kMaxChain];
    const float* bias[kMaxChain];
    int cin[kMaxChain], cout[kMaxChain], k[kMaxChain], act[kMaxChain];
    const void* res;  // residual added at the last layer, [N][H][W][Cout_last], nullable
    void* y;
    int N, H, W;
    int pool;  // 0 / 2 on the last layer
};

// Tiling of a chain chosen from the SM-count knob (Sec. IV-B: more cores -> smaller tiles ->
// more recomputed halo).
struct ChainTiling {
    int th, tw;          // output tile of the last layer (before pooling)
    int halo;            // sum of the layers' paddings
    int pitch, rows;     // frame of the input tile: (th + 2 halo) x (tw + 2 halo), pitch = width
    int tiles_h, tiles_w, n_tiles;
    int in_ring;         // 1: the first layer is 1x1 and its input planes stream through the slots one by one
    int in_group;        // input planes loaded side by side (one producer round)
    int in_slots;        // input plane slots in shared memory
    int out_mode;        // last layer: 0 direct 16-byte stores, 1 staging tile + TMA stores, 2 pooled out of a staging tile
    int stg_bufs;        // staging buffers (0 for direct stores)
    int stages;          // weight ring depth
    int stage_bytes;
    size_t smem_bytes;
    double redundancy;   // computed / useful multiply-accumulates
    double cost;         // the tiler's time estimate (SM clocks)
    bool ok;
};

int cuda_fail(cudaError_t e);  // records the error for dlf_last_cuda_error, returns DLF_E_CUDA
int cuda_fail_drv(int e);

// A kernel's shared-memory attribute belongs to a device, not to the process: the *_init functions keep one
// "done" flag per device, indexed by the current device.  -1: no current device or beyond the table.
constexpr int kMaxDevices = 64;
inline int current_device_slot() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

// Sets the kernels' shared-memory attributes once per device (outside any stream capture).
int kernels_init();
int conv_tc_init();
int chain_tc_init();

// Launches a kernel, optionally with programmatic dependent launch (the kernel must then call
// pdl_wait() before it touches anything its predecessor in the stream produces).
extern int g_use_pdl;
extern int g_conv_row_mode;  // conv_tc row mode: 0 never, 1 where it cuts the streamed bytes by a fifth, 2 wherever it applies
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(static_cast<unsigned>(block));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_use_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// kernels_mem.cu
int launch_conv_direct(const ConvArgs& a, int sm_count, cudaStream_t s);
int launch_dw3x3(const ConvArgs& a, int sm_count, cudaStream_t s);
int launch_maxpool(const void* x, void* y, int N, int H, int W, int C, int k, int stride, int pad, int Ho, int Wo,
                   int sm_count, cudaStream_t s);
int launch_gavgpool(const void* x, void* y, int N, int H, int W, int C, int sm_count, cudaStream_t s);
int launch_fc(const void* x, const void* w, const float* bias, void* y, int N, int K, int M, int act, int sm_count,
              cudaStream_t s);

int launch_stall(int* status_dev, unsigned long long limit_ns, cudaStream_t s);

// conv_tc.cu
bool conv_tc_supported(const ConvArgs& a);
bool chain_tc_layer_supported(int cin, int cout, int k);
int launch_conv_tc(const ConvArgs& a, int sm_count, int* status_dev, cudaStream_t s);
// Several layers as one persistent kernel with device-wide barriers between them (conv_tc.cu).
bool conv_seq_layer_supported(const ConvArgs& a);
int conv_seq_max_layers();
int launch_conv_seq(const ConvArgs* layers, int n_layers, int sm_count, int* status_dev, unsigned* sync_dev, cudaStream_t s);

// stem_tc.cu
bool stem_tc_supported(const ConvArgs& a);
int stem_tc_init();
int launch_stem_tc(const ConvArgs& a, int sm_count, int* status_dev, cudaStream_t s);

// mbconv_tc.cu: fused inverted-residual block (1x1 expansion, depthwise 3x3, 1x1 projection)
struct MbconvArgs {
    const void* x;           // [N][H][W][Cin]
    const void *w1, *wd, *w2;  // [hid][Cin], [hid][3][3][1], [Cout][hid]
    const float *b1, *bd, *b2;
    const void* res;         // [N][Ho][Wo][Cout] or null
    void* y;
    int N, H, W, Cin, hid, Cout, stride;
    int has_expand, act1, act2, act3;
};
struct MbconvTiling {
    int th, tw, fh, fw, nb1, nb2, tiles_h, tiles_w, n_tiles, stages, stage_bytes;
    int out_planes;  // 64-channel planes of the output staging buffer, 0 = none (direct stores)
    size_t smem_bytes;
    double redundancy;
    double cost;     // the tiler's time estimate (SM clocks)
    bool ok;
};
bool mbconv_supported(const MbconvArgs& a);
MbconvTiling mbconv_tiling(const MbconvArgs& a, int sm_count);
int mbconv_tc_init();
int launch_mbconv_tc(const MbconvArgs& a, const MbconvTiling& t, int sm_count, int* status_dev, cudaStream_t s);

// chain_tc.cu
ChainTiling chain_tc_tiling(const ChainArgs& a, int sm_count, int device_sms);
int launch_chain_tc(const ChainArgs& a, const ChainTiling& t, int sm_count, int* status_dev, cudaStream_t s);

// tensor map encoding through the driver entry point (no link-time dependency on libcuda)
int encode_tmap(void* out_map /*CUtensorMap*/, const void* base, int rank, const uint64_t* dims,
                const uint64_t* strides_bytes /*rank-1*/, const uint32_t* box, const uint32_t* elem_strides);

}  // namespace dlf
