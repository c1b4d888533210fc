/*
 * dlfusion.h - C ABI of the fused conv-group executor for NVIDIA B200 (sm_100a).
 *
 * A network is a list of layers.  A *plan* cuts the list into contiguous fusion groups and
 * gives each group a number of SMs: the two outputs of the paper's Algorithm 1
 * (fusion_partition_index[] and mp_of_fusionblock[]) and the two knobs of its Sec. II-A.2
 * ("model parallelism" = cores used by an operator or block, and "layer fusion").  A group
 * runs as one kernel whose intermediate feature maps stay in shared / tensor memory
 * (Sec. III-B: the output of a fused layer is produced on chip and reused at once); a
 * group's last layer is written to HBM.  All plans compute the same values: activations
 * are fp16, arithmetic is fp32, and every layer's result is rounded to fp16 once
 * (round-to-nearest-even) whether or not it leaves the chip.
 *
 * Conventions
 *   - Every call returns an int status: DLF_OK or a negative DLF_E_* code.  Nothing throws,
 *     aborts or exits.  dlf_strerror() names a code; dlf_last_cuda_error() returns the last
 *     CUDA runtime/driver error number seen by the calling thread's most recent failing call.
 *   - Pointers named *_dev are DEVICE pointers, *_host are HOST pointers; everything else
 *     (descriptors, plans, out-parameters) is host memory.
 *   - The caller owns all device memory: input, output, weights, biases and one workspace
 *     whose size the library reports.  The library allocates no device memory.  Device
 *     pointers are borrowed: they must stay valid until replaced or the net is destroyed.
 *   - Tensors are NHWC fp16 (IEEE binary16).  Weights are [cout][kh][kw][cin/groups] fp16
 *     (a fully connected layer: [cout][cin], cin in NHWC-flatten order).  Biases are fp32.
 *     Device pointers must be 16-byte aligned (256-byte for the workspace).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Calls on one dlf_net must not overlap in time; different nets are independent.
 */
#ifndef DLFUSION_H_
#define DLFUSION_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    DLF_OK = 0,
    DLF_E_INVALID_ARG = -1, /* null pointer, non-positive size, bad enum                        */
    DLF_E_SHAPE = -2,       /* layer list does not type-check (channels, empty output, src)     */
    DLF_E_PLAN = -3,        /* plan is not a contiguous cover, SM count out of range, or a group
                               cannot run as one kernel (never silently re-partitioned)         */
    DLF_E_WORKSPACE = -4,   /* workspace missing, misaligned or too small                       */
    DLF_E_UNSUPPORTED = -5, /* layer type / parameter combination has no kernel                 */
    DLF_E_CUDA = -6,        /* a CUDA call failed; see dlf_last_cuda_error()                    */
    DLF_E_TIMEOUT = -7,     /* a bounded device-side wait gave up (status word set by a kernel)  */
    DLF_E_STATE = -8        /* call out of order: weights or plan missing                       */
};

typedef enum { DLF_CONV = 0, DLF_DWCONV = 1, DLF_FC = 2, DLF_MAXPOOL = 3, DLF_GAVGPOOL = 4 } dlf_op;
typedef enum { DLF_ACT_NONE = 0, DLF_ACT_RELU = 1, DLF_ACT_RELU6 = 2 } dlf_act;

/* One layer, in the paper's {C_in, C_out, H_out x W_out, K_h x K_w} notation (Sec. II-B) plus
 * what the fused epilogue needs.  BatchNorm is folded into the bias. */
typedef struct {
    int32_t op;      /* dlf_op                                                                  */
    int32_t act;     /* dlf_act, applied after bias (and residual)                              */
    int32_t cin, cout;
    int32_t kh, kw, stride, pad;
    int32_t groups;  /* 1 = dense; cin for depthwise (DLF_DWCONV requires groups == cin == cout) */
    int32_t src;     /* index of the layer whose output this layer reads; -1 = network input    */
    int32_t res_src; /* -2 = none; -1 = network input; else layer index added before the act.   */
    int32_t pool;    /* 0, or 2 = 2x2 stride-2 max-pool fused after the activation              */
} dlf_layer_desc;

/* Parameters of Eq. 5 and Algorithm 1.  Eq. 5 gives a proportionality only, so the per-layer SM
 * count is clamp(round(kappa * (alpha*log2(C_out) + beta*log2(ops)) + kappa0), 1, s_max), with
 * ops = Eq. 1 / Eq. 2 times the batch and divided by the groups.  op_critical is Algorithm 1's
 * OpCount_critical in the same unit (operations per SM). */
typedef struct {
    double alpha, beta;   /* paper's MLU100 values: 0.316, 0.659                                 */
    double kappa, kappa0; /* affine map from the Eq. 5 score to an SM count                      */
    double op_critical;   /* close a block when sum_ops / avg_sm >= op_critical                  */
    int32_t s_max;        /* largest SM count (<= SMs of the device); 0 = all SMs                */
    int32_t legalise;     /* 0: pure Algorithm 1 (blocks close only where no kernel could ever
                             fuse across: structural rule).  1: also split blocks the fused
                             kernel cannot hold (shared / tensor memory capacity)                */
} dlf_tuner_params;

/* Reduced brute-force search (paper Sec. V, "Oracle Case"): every candidate group (a legal span
 * of at most max_group_len layers, one SM count out of sm_choices) is timed once on the device
 * and the best contiguous partition is found by dynamic programming over the measured times. */
typedef struct {
    int32_t n_sm_choices;
    int32_t sm_choices[16];
    int32_t max_group_len;
    int32_t warmup, iters;
} dlf_search_params;

typedef struct dlf_net dlf_net;

const char* dlf_strerror(int status);
int dlf_last_cuda_error(void);
/* Number of SMs of the current device (the upper limit of the SM-count knob), or a DLF_E_* code. */
int dlf_device_sm_count(void);

/* Builds a net from n_layers descriptors (copied) for an N x H x W x C fp16 NHWC input.
 * Infers every layer's output shape, H_out = floor((H + 2 pad - k) / stride) + 1, and its
 * operation count (Eq. 1 / Eq. 2).  Errors: DLF_E_INVALID_ARG, DLF_E_SHAPE, DLF_E_UNSUPPORTED. */
int dlf_net_create(const dlf_layer_desc* layers, int n_layers, int N, int H, int W, int C,
                   dlf_net** out);
void dlf_net_destroy(dlf_net* net);

/* ops_eq1: Eq. 1 / Eq. 2 exactly as printed (no batch, no groups; this is what reproduces the
 * paper's Table 2).  flops: useful operations of one run (batch included, divided by groups).
 * out_shape: {N, H, W, C}.  Any out-pointer may be NULL. */
int dlf_net_layer_info(const dlf_net* net, int layer, int64_t* ops_eq1, int64_t* flops,
                       int64_t out_shape[4]);

/* Device pointers to one layer's weights and bias (borrowed).  Layers without parameters
 * (pools) take none.  Changing weights invalidates nothing else. */
int dlf_net_set_weights(dlf_net* net, int layer, const void* w_f16_dev, const float* bias_dev);

/* Workspace: staging for the input of dlf_net_run_host, one slot per layer output (the worst
 * case over plans is the unfused plan, where every layer reaches HBM), scratch for split
 * reductions (fp32 partial tiles and their arrival counters, which bind_workspace zeroes and
 * every launch leaves at zero) and a status word.  Contents are undefined between runs; runs of
 * one net must not overlap in time (they share the slots and the scratch). */
int dlf_net_workspace_bytes(const dlf_net* net, size_t* bytes);
int dlf_net_bind_workspace(dlf_net* net, void* workspace_dev, size_t bytes);

/* Sets the plan: group g covers layers (group_end[g-1], group_end[g]] (inclusive end index) and
 * runs on sm_count[g] SMs (a persistent grid of that many CTAs).  DLF_E_PLAN if the ends are not
 * strictly increasing up to n_layers-1, an SM count is outside [1, #SMs], or a group with more
 * than one layer is not a chain the fused kernel can hold. */
int dlf_net_set_plan(dlf_net* net, int n_groups, const int32_t* group_end, const int32_t* sm_count);
/* The no-fusion plan: one group per layer, all SMs. */
int dlf_net_plan_unfused(dlf_net* net);
/* Reads back the current plan; arrays must hold n_layers entries. */
int dlf_net_get_plan(const dlf_net* net, int* n_groups, int32_t* group_end, int32_t* sm_count);
/* 1 if layers first..last can run as one fused kernel on `sm_count` SMs, 0 if not. */
int dlf_net_group_is_legal(const dlf_net* net, int first, int last, int sm_count);

/* The rule that bounds Algorithm 1's blocks here (the paper's vendor SDK fuses "almost arbitrary" layers, Sec. III-B; this
 * library has four fused kernels): 1 if the tuner may propose layers first..last as one group on s_max SMs - the span is
 * an inverted-residual block or a dense chain whose fused kernel is estimated (by its own tiler) to beat one kernel per
 * layer, or a residual block's 1x1 projection branch followed by the 1x1 expansion layer it is added to (one product whose
 * K runs over both inputs: the projection's value joins the fp32 sum without a rounding of its own, at most half an fp16
 * unit in the last place of that value away from the layer-by-layer result), or, with DLF_OPT_GROUP_KERNEL = 2, any run of
 * dense convolutions.  With prefix != 0
 * the layers may also be the beginning of an inverted-residual block that can still grow.  0 if not.  Host only. */
int dlf_net_tuner_may_fuse(const dlf_net* net, int first, int last, int prefix, int s_max);

/* Algorithm 1 with Eq. 5 (host only, O(n)).  Writes the plan into the arrays (n_layers entries
 * each) and does NOT install it; pass it to dlf_net_set_plan. */
int dlf_net_autotune(const dlf_net* net, const dlf_tuner_params* params, int* n_groups,
                     int32_t* group_end, int32_t* sm_count);

/* Reduced brute-force search; needs weights and workspace.  Installs nothing; leaves the net's
 * plan as it was.  best_ms: the dynamic programme's optimum (sum of group times). */
int dlf_net_bruteforce(dlf_net* net, const dlf_search_params* params, const void* in_dev,
                       void* stream, int* n_groups, int32_t* group_end, int32_t* sm_count,
                       float* best_ms);

/* The search's dynamic programme alone, on a table the caller supplies (host only; no net, no device): ms is
 * [n_layers][max_group_len][n_sm_choices], the time of span a..a+len-1 on sm_choices[c] SMs at
 * ms[(a * max_group_len + len - 1) * n_sm_choices + c], negative for a group that cannot run.  Returns the contiguous
 * partition with the least total time (Sec. V: a plan's time is the sum of its blocks' times), each group with the SM
 * count that gave its best time.  DLF_E_PLAN if no partition is possible. */
int dlf_bruteforce_table(int n_layers, int max_group_len, int n_sm_choices, const int32_t* sm_choices, const float* ms,
                         int* n_groups, int32_t* group_end, int32_t* sm_count, float* best_ms);

/* Times layers first..last as ONE candidate group on sm_count SMs, outside any plan (the single-layer
 * micro-benchmark of the paper's characterisation, Sec. II-B, and one cell of the reduced brute-force
 * search, Sec. V): median device time of one launch, taken over `iters` timings of four back-to-back
 * launches after `warmup` untimed ones (warm L2).  The group reads its inputs from the workspace slots
 * of the layers before it: with prepare != 0 the call first runs the no-fusion plan once to fill every
 * slot (the installed plan is kept); with prepare == 0 the caller has done so.  DLF_E_PLAN if the span
 * cannot run as one kernel on that many SMs.  The network's last layer is written to its workspace slot. */
int dlf_net_time_span(dlf_net* net, int first, int last, int sm_count, const void* in_dev, void* stream,
                      int warmup, int iters, int prepare, float* ms);

/* Enqueues one inference on `stream` and returns without waiting.  in_dev: N*H*W*C fp16.
 * out_dev: the last layer's output, fp16 NHWC.  DLF_E_STATE without weights / plan /
 * workspace. */
int dlf_net_run(dlf_net* net, const void* in_f16_dev, void* out_f16_dev, void* stream);
/* Same with HOST buffers: copies the input to the device, runs, copies the output back and
 * waits for the stream.  For asynchronous copies the host buffers should be page-locked. */
int dlf_net_run_host(dlf_net* net, const void* in_f16_host, void* out_f16_host, void* stream);
/* Waits for the stream and reports a device-side bounded wait that gave up (DLF_E_TIMEOUT)
 * or a CUDA error from the kernels enqueued so far. */
int dlf_net_sync(dlf_net* net, void* stream);

/* Self-test of the bounded device-side waits: enqueues a one-CTA kernel that waits - through the very routine every kernel's
 * waits use - at a barrier nothing arrives at, with the limit lowered from one second to limit_us microseconds.  The wait
 * gives up, records its code in the net's status word and the kernel ends normally; the next dlf_net_sync on that stream
 * returns DLF_E_TIMEOUT (and clears the word), later runs are unaffected.  Nothing traps, nothing spins beyond the limit. */
int dlf_net_debug_stall(dlf_net* net, int limit_us, void* stream);

/* Times `iters` runs with CUDA events on `stream` after `warmup` untimed ones.  If flush_dev is
 * non-NULL its flush_bytes are overwritten before every run, outside the timed interval, to
 * evict L2.  ms_median / ms_min: per-run times.  ms_per_group (may be NULL): median time of
 * each group from a second, instrumented pass with an event after every group. */
int dlf_net_time(dlf_net* net, const void* in_dev, void* out_dev, void* stream, int warmup,
                 int iters, void* flush_dev, size_t flush_bytes, float* ms_median, float* ms_min,
                 float* ms_per_group);

/* Device pointer and shape of a layer output that the current plan writes to HBM (a group's
 * last layer); valid after a run.  DLF_E_PLAN for a layer inside a group. */
int dlf_net_boundary_tensor(const dlf_net* net, int layer, const void** dev_ptr, int64_t shape[4]);

/* Roofline model of group g of the current plan: useful flops, compulsory HBM bytes (the
 * group's external inputs once, its output, its weights and biases once; maps inside the group
 * count zero, Eq. 3 applied to the group), the ratio computed/useful multiply-accumulates
 * including the recomputed halo of the chosen tiling (Sec. IV-B), and the number of kernels the
 * group launches. */
int dlf_net_group_model(const dlf_net* net, int group, int64_t* flops, int64_t* hbm_bytes,
                        double* redundancy, int* launches);

/* Name of the kernel variant that runs group g ("chain_tc", "conv_seq", "mbconv_tc", "conv_tc", "stem_tc",
 * "conv_direct", "dw3x3", "fc", "maxpool", "gavgpool"); the string is owned by the library. */
const char* dlf_net_group_kernel(const dlf_net* net, int group);

/* Options (debugging and ablation); setting one clears the plan, which must be set again.
 *   DLF_OPT_NO_TENSOR_CORE   1: route every dense convolution to the CUDA-core direct kernel
 *                               (multi-layer groups then become illegal).
 *   DLF_OPT_SINGLE_AS_CHAIN  1: a single stride-1 1x1 / 3x3 convolution with <= 256 output
 *                               channels runs through the fused-chain kernel (input tile
 *                               loaded once) instead of the per-tap kernel.
 *   DLF_OPT_GROUP_KERNEL     which kernel runs a multi-layer group of dense convolutions.  0 (default): narrow stride-1
 *                               1x1 / 3x3 chains (at most 64 channels) are handed over tile by tile in shared memory, every
 *                               other run of dense convolutions layer by layer through L2 inside one persistent kernel
 *                               (device-wide barrier between layers); 1: shared memory wherever the chain kernel can hold
 *                               the group; 2: L2 wherever possible.
 *   DLF_OPT_CUDA_GRAPH       1 (default): dlf_net_run replays one CUDA graph that holds every
 *                               group of the plan (captured on the first run and whenever the
 *                               input / output pointers, weights, workspace or plan change);
 *                               0: launch the kernels one by one.  Does not clear the plan.
 *   DLF_OPT_PDL              1 (default): the tensor-core kernels are launched with programmatic
 *                               dependent launch, so that a kernel's set-up overlaps the tail of
 *                               its predecessor; 0: plain stream order.  Process-wide.
 *   DLF_OPT_CONV_ROW_MODE    1 (default): a single 3x3 stride-1 convolution whose C_in is a multiple of 64 and
 *                               whose image is at most 126 pixels wide loads a kernel row's input window once for
 *                               its three taps where that cuts the bytes a CTA streams by a fifth; 0: never (one
 *                               window load per tap); 2: wherever it applies.  Process-wide; does not clear the plan. */
enum { DLF_OPT_NO_TENSOR_CORE = 1, /* 2 is unused */ DLF_OPT_SINGLE_AS_CHAIN = 3, DLF_OPT_CUDA_GRAPH = 4, DLF_OPT_PDL = 5,
       DLF_OPT_CONV_ROW_MODE = 6, DLF_OPT_GROUP_KERNEL = 7 };
int dlf_net_set_option(dlf_net* net, int option, int value);

/* Size of the scratch array that dlf_conv_chain_run_static keeps inside the library image. */
#define DLF_STATIC_SCRATCH_BYTES (16u << 20)

/* (The paper has no counterpart for this call.)
 *
 * Runs a chain of 1..8 dense convolutions (DLF_CONV, groups 1, no residual, no fused pool; layer i
 * reads layer i-1, layer 0 reads x), one tensor-core kernel per layer, WITHOUT a workspace and
 * without allocating anything: the maps between the layers and the kernels' status word live in
 * a fixed DLF_STATIC_SCRATCH_BYTES (16 MiB) array that is part of the library and therefore
 * occupies that much memory on every GPU that loads it, until the process exits.
 *
 * It is meant for callers that must not, or cannot, call cudaMalloc: code running between other
 * frameworks that have already claimed the whole device, services with a fixed memory budget
 * decided at start-up, and latency-critical loops in which an allocation's implicit device-wide
 * synchronisation is unacceptable.  The caller still owns x, the weights, the biases and y.
 *
 *   layers[i].src must be i-1; cin, cout multiples of 8; stride 1 or 2.
 *   w_f16_dev[i], bias_dev[i]: device pointers, layouts as for dlf_net_set_weights.
 *   y_f16_dev: the last layer's output, fp16 NHWC.
 *   sm_count: persistent grid size of every kernel (1 .. SMs of the device).
 *
 * Limits and errors: every map BETWEEN two layers must fit in half of the array (8 MiB), else
 * DLF_E_WORKSPACE and nothing is enqueued; DLF_E_SHAPE / DLF_E_UNSUPPORTED / DLF_E_INVALID_ARG as
 * for dlf_net_create.  The call enqueues on `stream`, waits for it, and returns DLF_E_TIMEOUT if
 * a kernel's bounded wait gave up.
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current); make that first call before starting any stream capture.  All calls
 * share the one array: it still holds the previous call's maps, the status word is cleared at
 * the start of every call, and two calls that overlap on the same GPU (different streams or
 * threads) overwrite each other's intermediate maps - run them one after another. */
int dlf_conv_chain_run_static(const dlf_layer_desc* layers, int n_layers, int N, int H, int W,
                              const void* x_f16_dev, const void* const* w_f16_dev,
                              const float* const* bias_dev, void* y_f16_dev, int sm_count, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DLFUSION_H_ */
