// dlf_conv_chain_run_static: a chain of dense convolutions, one kernel per layer, whose scratch
// memory (the maps between the layers and the kernels' status word) is a fixed array inside the
// library image instead of a caller-provided workspace.  The paper has no counterpart; the entry
// point exists for callers that cannot allocate device memory.
#include <cuda_runtime.h>

#include <cstring>
#include <mutex>

#include "internal.h"

namespace {

// Two halves for the ping-pong between layers, then the status word.
constexpr size_t kHalfBytes = DLF_STATIC_SCRATCH_BYTES / 2;
static __device__ __align__(256) unsigned char g_static_scratch[DLF_STATIC_SCRATCH_BYTES + 256];

unsigned char* g_scratch_addr[dlf::kMaxDevices];  // device address of the array, per device, once resolved
std::mutex g_scratch_mutex;                  // guards the table above

// In host code `g_static_scratch` is only a handle for the symbol, not a device address: the
// address a kernel can use has to be asked for, with the device in question current.
int scratch_address(unsigned char** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return dlf::cuda_fail(e);
    if (dev < 0 || dev >= dlf::kMaxDevices) return DLF_E_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return dlf::cuda_fail(e);
        g_scratch_addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_addr[dev];
    return DLF_OK;
}

}  // namespace

extern "C" int dlf_conv_chain_run_static(const dlf_layer_desc* layers, int n_layers, int N, int H, int W,
                                         const void* x_f16_dev, const void* const* w_f16_dev,
                                         const float* const* bias_dev, void* y_f16_dev, int sm_count, void* stream) {
    using namespace dlf;
    if (!layers || !x_f16_dev || !w_f16_dev || !bias_dev || !y_f16_dev) return DLF_E_INVALID_ARG;
    if (n_layers < 1 || n_layers > kMaxChain || N < 1 || H < 1 || W < 1 || sm_count < 1) return DLF_E_INVALID_ARG;
    // shapes first: nothing is enqueued unless every layer fits
    ConvArgs a[kMaxChain];
    int h = H, w = W;
    for (int i = 0; i < n_layers; i++) {
        const dlf_layer_desc& d = layers[i];
        if (d.op != DLF_CONV || d.groups != 1 || d.res_src != -2 || d.pool != 0) return DLF_E_UNSUPPORTED;
        if (d.act < DLF_ACT_NONE || d.act > DLF_ACT_RELU6) return DLF_E_INVALID_ARG;
        if (d.cin < 8 || d.cout < 8) return DLF_E_SHAPE;
        if (d.src != i - 1 || (i > 0 && d.cin != layers[i - 1].cout)) return DLF_E_SHAPE;
        if (d.kh < 1 || d.kw < 1 || d.stride < 1 || d.pad < 0 || h + 2 * d.pad < d.kh || w + 2 * d.pad < d.kw) return DLF_E_SHAPE;
        if (!w_f16_dev[i] || !bias_dev[i]) return DLF_E_INVALID_ARG;
        ConvArgs& c = a[i];
        std::memset(&c, 0, sizeof(c));
        c.N = N; c.H = h; c.W = w; c.Cin = d.cin; c.Cout = d.cout;
        c.Ho = (h + 2 * d.pad - d.kh) / d.stride + 1;
        c.Wo = (w + 2 * d.pad - d.kw) / d.stride + 1;
        c.kh = d.kh; c.kw = d.kw; c.stride = d.stride; c.pad = d.pad; c.groups = 1; c.act = d.act; c.pool = 0;
        c.w = w_f16_dev[i];
        c.bias = bias_dev[i];
        if (!conv_tc_supported(c)) return DLF_E_UNSUPPORTED;
        const size_t out_bytes = static_cast<size_t>(N) * c.Ho * c.Wo * d.cout * 2;
        if (i < n_layers - 1 && out_bytes > kHalfBytes) return DLF_E_WORKSPACE;  // intermediate map beyond the fixed scratch
        h = c.Ho;
        w = c.Wo;
    }
    int rc = conv_tc_init();
    if (rc) return rc;
    unsigned char* scratch = nullptr;
    rc = scratch_address(&scratch);
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int* status = reinterpret_cast<int*>(scratch + DLF_STATIC_SCRATCH_BYTES);
    // the array keeps what the previous call left: the status word has to start at zero
    cudaError_t e = cudaMemsetAsync(status, 0, sizeof(int), s);
    if (e != cudaSuccess) return cuda_fail(e);
    for (int i = 0; i < n_layers; i++) {
        a[i].x = i == 0 ? x_f16_dev : scratch + ((i - 1) & 1) * kHalfBytes;
        a[i].y = i == n_layers - 1 ? y_f16_dev : static_cast<void*>(scratch + (i & 1) * kHalfBytes);
        rc = launch_conv_tc(a[i], sm_count, status, s);
        if (rc) return rc;
    }
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e);
    int st = 0;
    e = cudaMemcpy(&st, status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    return st == 0 ? DLF_OK : DLF_E_TIMEOUT;
}
