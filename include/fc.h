/*
 * fc.h -- C ABI of the fused-chain library for NVIDIA B200 (sm_100a).
 *
 * A "chain" is what the paper's agent produces when it fuses a PyTorch operator sequence into
 * one CUDA kernel (composed-operator problems, "Level 2"; the paper's fusion rationale is to
 * remove global-memory round trips and extra launches between a producer and its epilogue):
 *
 *     producer  ->  ordered elementwise epilogue ops  ->  optional row / channel reduction
 *
 *   producer   ELEMENTWISE  v[m][n] = x[m][n]
 *              GEMM_NT      v[m][n] = sum_k A[m][k] * B[n][k]          (B stored [N x K] row-major,
 *                           the "weight is [out_features x in_features]" convention of the paper's
 *                           appendix GEMM / linear-layer kernels), fp32 accumulation
 *              CONV2D_NHWC  v[b][oh][ow][co] = sum_{r,s,ci} in[b][oh*stride-pad+r][ow*stride-pad+s][ci]
 *                           * W[co][r][s][ci]   (cross-correlation, zero padding, floor output size,
 *                           as in the paper's appendix convolution kernel; layout restated for NHWC)
 *              CONV2D_NCHW  the same sum on the appendix kernel's own layouts, in[b][ci][h][w] and
 *                           W[co][ci][r][s]; outputs are the pooled ones, unchanged
 *   ops        bias over the last index, per-column affine, ReLU, tanh-GELU, scalar scale, clamp,
 *              add a tensor of the output's shape (bias -> ReLU -> scale is the paper's appendix
 *              epilogue; the others are named by this repository's benchmark configurations)
 *   reduction  row logsumexp (its size-one case is the identity the paper's Q18 analysis uses),
 *              row softmax, global average pool over (oh, ow)
 *
 * Ownership.  Every tensor and the workspace are allocated and freed by the caller.  fc_run never
 * allocates device memory and never synchronises; it enqueues at most two memsets and one to four
 * kernels on the given stream (one more in front of a few-channel convolution that runs on a bordered copy
 * of its image, see fc_workspace_size_split) and returns (two kernels: a convolution behind the kernel that zeroes
 * its pooled output -- not launched for a 2x2 max-pool over tiles of whole row pairs, which stores every
 * window once --, or a wide GEMM + ROW_SOFTMAX as the GEMM kernel and a rescaling pass; three: the
 * collapsed linear layer; four: CONV2D_NCHW with its two layout kernels).  Inputs are read-only;
 * outputs are fully overwritten.
 *
 * Launches.  Kernels are launched with programmatic stream serialization and wait, before their first access to
 * global memory, for everything in front of them in the stream: the order the caller sees is the stream's,
 * only launch latency overlaps the tail of the work in front.  Calls may be captured into a CUDA graph.
 *
 * Pointers.  Unless a function says "host", every fc_tensor.ptr is a DEVICE pointer.
 *
 * Layout.  Row-major contiguous only (stride[] must describe exactly that, in elements).
 *   GEMM_NT: inputs[0] = A [M,K], inputs[1] = B [N,K].  CONV2D_NHWC: inputs[0] = image
 *   [batch,H,W,Cin], inputs[1] = weights [Cout,R,S,Cin].  CONV2D_NCHW: inputs[0] = image [batch,Cin,H,W],
 *   inputs[1] = weights [Cout,Cin,R,S].  ELEMENTWISE: inputs[0] = x [M,N].
 *   Further inputs are the vectors ([N] or [Cout]) and tensors that fc_op.in0 / in1 index.
 *   Outputs, in order: the main output (if store_main, or if reduce == ROW_SOFTMAX, whose
 *   probabilities take the main output's place), then the reduction (LOGSUMEXP / ROW_SUM / ROW_MAX /
 *   ROW_MEAN: f32 [M];
 *   GLOBAL_AVGPOOL: f32 [batch,Cout]).
 *
 * Alignment.  Base pointers of bf16 / fp16 operands of GEMM / CONV must be 16-byte aligned and K (GEMM)
 * or Cin (CONV) a multiple of 8; violations return FC_ERR_ALIGNMENT.  Other tensors need only the
 * natural alignment of their element type (vector access is used when 16-byte alignment holds).
 *
 * Errors.  Return code only: nothing is thrown or printed, the process is never aborted.  Chains
 * outside the supported patterns return FC_ERR_UNSUPPORTED; there is no CPU fallback and no other
 * backend.  A device that is not compute capability 10.x returns FC_ERR_ARCH.  Device-side waits
 * are bounded; if one expires the kernel records FC_ERR_TIMEOUT in a device status word, skips its
 * remaining stores and exits; fc_get_async_status reports it.  A launch that gave up may leave its
 * cross-tile counters (in the workspace) at a non-zero count, and only fc_get_async_status puts them
 * back: after any fc_run that can have timed out, read the status before the next fc_run on that
 * device, or the next chain that uses the workspace may skip its waits and store wrong values.
 *
 * Testing aid.  fc_testing_set (end of this file) flips switches that exist for the test suite only: one makes
 * the cross-tile wait of GEMM_NT + ROW_SOFTMAX launches expect an arrival that never comes, so that the bounded
 * wait expires (about two seconds), nothing is stored, and fc_get_async_status returns FC_ERR_TIMEOUT while the
 * device stays usable; the other does the same to the wait of a split tile's merging slice.
 *
 * Debug build.  The same sources compiled with -DFC_DEBUG (paper_2602_14293_b200/build.py builds it as libfc_debug.so)
 * check, in the kernels, every global-memory address that comes out of their own index arithmetic (output stores of
 * the tensor-core epilogues, split-tile scratch, statistics, pooled atomics, the elementwise kernels' loads and
 * stores) against the extent of the tensor it belongs to.  A failed check skips the access and records
 * FC_ERR_BOUNDS with a site number in the device status word; nothing traps.  FC_TESTING_BOUNDS_TRIP makes such a
 * build believe that the main output is one row shorter than it is, to show the mechanism at work.
 *
 * Threading.  fc_run may be called from several host threads.  The workspace set by
 * fc_set_workspace is shared by all calls: launches that use it (row reductions on a GEMM, CONV2D_NCHW) must not
 * overlap on the device.
 */
#ifndef FC_H_
#define FC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FC_VERSION 2    /* 2: FC_MAX_OPS 8 -> 12 (a four-layer chain with bias and activation needs ten ops) */
#define FC_MAX_OPS 12

typedef enum {
    FC_OK = 0,
    FC_ERR_NULL = 1,          /* a required pointer is null                                   */
    FC_ERR_INVALID_SPEC = 2,  /* struct_size / version / enum value / op operand index wrong  */
    FC_ERR_UNSUPPORTED = 3,   /* well-formed chain that no kernel here implements             */
    FC_ERR_SHAPE = 4,         /* a dimension < 1, or a tensor's shape does not fit the spec   */
    FC_ERR_ALIGNMENT = 5,
    FC_ERR_WORKSPACE = 6,     /* chain needs a workspace and none (or too small) was set      */
    FC_ERR_ARCH = 7,
    FC_ERR_CUDA = 8,          /* a CUDA runtime / driver call failed; see fc_last_error       */
    FC_ERR_TIMEOUT = 9,       /* a bounded device-side wait expired                           */
    FC_ERR_BOUNDS = 10        /* debug build (libfc_debug.so, compiled with -DFC_DEBUG) only: an address that a kernel
                                 computed for one of its tensors lay outside that tensor; the access was skipped and
                                 fc_get_async_status reports this code (fc_last_error names the site)              */
} fc_status;

typedef enum {
    FC_F32 = 0,       /* as spec.in_dtype of a GEMM_NT producer: fp32 operands, fp32 output, no reduction.  Small problems
                         (M N K < 2^29) are contracted with fp32 FMAs on the plain ALUs.  Larger ones run on the tensor
                         cores when K is a multiple of 4, both operands are 16-byte aligned and a workspace of
                         roundup(12 M K, 256) + 12 N K bytes is registered (fc_workspace_size reports it): every operand
                         value x is cut into hi (the bits a tf32 multiplication reads) and lo = x - hi, and
                         A B^T = A_hi B_hi^T + A_hi B_lo^T + A_lo B_hi^T with fp32 accumulation, which leaves out terms of
                         2^-21 relative size per product.  Without the workspace the fp32-FMA kernels run at any size. */
    FC_BF16 = 1,
    FC_F16 = 2,       /* IEEE binary16, the storage type of the paper's kernels */
    FC_F8E4M3 = 3,    /* 8-bit float, 4 exponent bits (bias 7), 3 fraction bits, finite only (no infinities, all-ones is NaN):
                         storage of BOTH operands of a GEMM_NT producer (fp32 accumulation on the tensor cores, K a multiple
                         of 16); per-tensor scaling is the caller's, undone by a SCALE op.  Not an output, vector or
                         residual type, not for ELEMENTWISE / CONV producers or LINEAR ops. */
    FC_MXF8E4M3 = 4,  /* spec.in_dtype only: block-scaled 8-bit operands (the open "microscaling" format MXFP8 that the B200
                         tensor cores implement; the paper mentions 8-bit floats only in passing).  GEMM_NT with reduce NONE:
                         inputs[0] = A [M,K] and inputs[1] = B [N,K] are FC_F8E4M3 tensors, inputs[2] = SA [M, K/32] and
                         inputs[3] = SB [N, K/32] are FC_E8M0 tensors, and
                           v[m][n] = sum_j 2^(SA[m][j] - 127) 2^(SB[n][j] - 127) sum_{k = 32 j .. 32 j + 31} A[m][k] B[n][k].
                         K a multiple of 128, all four tensors 16-byte aligned.  The scales are first rewritten into the
                         tensor cores' tile order in the workspace (two small launches; fc_workspace_size reports the bytes:
                         (ceil(M/128) + 2 ceil(N/240)) * K/128 * 512, for N <= 128: (ceil(M/128) + 1) * K/128 * 512).  Ops and outputs as for the other 8-bit GEMM; vector and
                         tensor operands of ops are inputs[4..]. */
    FC_E8M0 = 5       /* a scale of FC_MXF8E4M3: one byte e meaning 2^(e - 127); 255 is NaN and must not occur */
} fc_dtype;

typedef enum {
    FC_PROD_ELEMENTWISE = 0,
    FC_PROD_GEMM_NT = 1,
    FC_PROD_CONV2D_NHWC = 2,
    FC_PROD_CONV2D_NCHW = 3   /* image [batch,Cin,H,W], weights [Cout,Cin,R,S]: both are first rewritten channels-last into
                                 the workspace (two transposition launches, fc_workspace_size reports the bytes: one copy
                                 of each), then the CONV2D_NHWC kernel runs on the copies.  Same limits as CONV2D_NHWC. */
} fc_producer;

typedef enum {
    FC_OP_BIAS_N = 0,     /* v += vec[in0][n]                      n = last (column / channel) index */
    FC_OP_AFFINE_N = 1,   /* v  = v * vec[in0][n] + vec[in1][n]                                      */
    FC_OP_RELU = 2,       /* v  = v < 0 ? 0 : v                                                      */
    FC_OP_GELU_TANH = 3,  /* v  = 0.5 v (1 + tanh(sqrt(2/pi) (v + 0.044715 v^3)))                    */
    FC_OP_SCALE = 4,      /* v *= f0                                                                 */
    FC_OP_CLAMP = 5,      /* v  = min(max(v, f0), f1)                                                */
    FC_OP_ADD_TENSOR = 6, /* v += tensor[in0][m][n]              same shape as the main output; may hold -inf (an additive
                             mask): ROW_SOFTMAX gives such entries exactly 0 and ROW_LOGSUMEXP ignores them; a row of -inf
                             only has no softmax (NaN, as the definition gives)                       */
    FC_OP_LINEAR = 7      /* v[m][:] = round16(v[m][:]) W^T, W = inputs[in0] of shape [N_next][N] in the chain's 16-bit
                             type: another linear layer.  The row is rounded to that type first (it is the tensor-core
                             operand, and what an unfused sequence would have stored); N becomes N_next for the ops
                             that follow.  16-bit GEMM_NT producer only, reduce NONE, every width (N and each N_next)
                             <= 256 so that a block of rows stays on chip and, except the last, a multiple of 8; at most three LINEAR
                             ops, no ADD_TENSOR: consecutive layers of the paper's appendix network                 */
} fc_op_kind;

typedef enum {
    FC_RED_NONE = 0,
    FC_RED_ROW_LOGSUMEXP = 1,   /* out[m] = max_n v + log sum_n exp(v - max)          */
    FC_RED_ROW_SOFTMAX = 2,     /* p[m][n] = exp(v - max) / sum_n exp(v - max)         (elementwise or GEMM producer) */
    FC_RED_GLOBAL_AVGPOOL = 3,  /* out[b][c] = mean over (oh, ow) of v[b][oh][ow][c]   */
    FC_RED_ROW_SUM = 4,         /* out[m] = sum_n v          (elementwise or GEMM producer) */
    FC_RED_ROW_MAX = 5,         /* out[m] = max_n v          (elementwise or GEMM producer) */
    FC_RED_ROW_MEAN = 6,        /* out[m] = (sum_n v) / N    (elementwise or GEMM producer) */
    FC_RED_MAXPOOL_2X2 = 7      /* out[b][i][j][c] = max of v[b][2i..2i+1][2j..2j+1][c], [batch][OH/2][OW/2][Cout];
                                   CONV producer whose op list ends with RELU (the conv / ReLU / max-pool stage
                                   of the paper's appendix network); a last odd row or column is dropped.
                                   Stored as fp32, or as out_dtype when that is FC_BF16 or FC_F16 (the next
                                   layer's operand type, the maximum rounded to nearest even): that form needs
                                   OH even and OW <= 64, else FC_ERR_UNSUPPORTED                              */
} fc_reduce;

typedef struct {
    int32_t kind;      /* fc_op_kind                       */
    int32_t in0, in1;  /* indices into inputs[] (unused: 0) */
    float f0, f1;
} fc_op;

typedef struct {
    uint32_t struct_size;   /* sizeof(fc_chain_spec) */
    uint32_t version;       /* FC_VERSION            */
    int32_t producer;       /* fc_producer           */
    int32_t in_dtype;       /* storage of inputs[0] (and inputs[1] for GEMM / CONV) */
    int32_t acc_dtype;      /* FC_F32                */
    int32_t out_dtype;      /* storage of the main output / softmax probabilities / a 2x2 max-pool (16-bit types) */
    int64_t M, N, K;        /* ELEMENTWISE: M rows x N cols; GEMM: M x N x K        */
    int64_t batch, H, W, Cin, Cout, R, S, stride, pad;   /* CONV only              */
    int32_t n_ops;
    fc_op ops[FC_MAX_OPS];  /* applied in order      */
    int32_t reduce;         /* fc_reduce             */
    int32_t store_main;     /* also write the main output when a reduction exists   */
} fc_chain_spec;

typedef struct {
    void* ptr;
    int32_t dtype;          /* fc_dtype */
    int32_t rank;
    int64_t shape[4];
    int64_t stride[4];      /* in elements; must be the contiguous row-major strides */
} fc_tensor;

/*
 * Run one fused chain: the whole operator sequence described by `spec` in one pass over the data
 * (the paper's fused-kernel launch, with raw pointers plus sizes as in its harness convention).
 * All tensor pointers are device pointers on the current device; `cuda_stream` is a cudaStream_t
 * (NULL = the legacy default stream).  Asynchronous.  Returns FC_OK once the work is enqueued.
 */
fc_status fc_run(const fc_chain_spec* spec, const fc_tensor* inputs, int n_inputs,
                 fc_tensor* outputs, int n_outputs, void* cuda_stream);

/*
 * Same chain with HOST buffers: every inputs[i].ptr / outputs[i].ptr is a host pointer (pinned
 * memory makes the copies asynchronous).  `staging` is a caller-owned DEVICE buffer of at least
 * fc_staging_size() bytes into which inputs are copied (cudaMemcpyAsync on the stream), the chain
 * runs there, and outputs are copied back.  Enqueues only; the caller synchronises the stream
 * before reading the outputs.  Chains that move 32 MB or more are cut into up to 8 row (image)
 * chunks whose copies run on two internal copy streams (created on the first such call on a
 * device), so that copy-in, kernel and copy-out of neighbouring chunks overlap; the work is still
 * ordered after everything enqueued on `cuda_stream` before the call, and `cuda_stream` waits for
 * the last copy-out.
 */
fc_status fc_run_host(const fc_chain_spec* spec, const fc_tensor* host_inputs, int n_inputs,
                      fc_tensor* host_outputs, int n_outputs, void* staging, size_t staging_bytes,
                      void* cuda_stream);
fc_status fc_staging_size(const fc_chain_spec* spec, const fc_tensor* inputs, int n_inputs,
                          const fc_tensor* outputs, int n_outputs, size_t* bytes);

/*
 * Scratch memory.  A 16-bit GEMM_NT with a row reduction needs some (per-tile partial results plus
 * per-panel arrival counters for the cross-tile merge; K + 1 doubles for the collapsed form, below), and so
 * does CONV2D_NCHW (the channels-last copies of image and weights).  The partial results are kept per row
 * and output tile; tiles are 128, 240 or 256 columns wide, whichever the launcher expects to be faster for the
 * shape, so a row reduction's value depends on the row count of the call up to fp32 summation order.
 * fc_workspace_size reports
 * the bytes a spec needs (0 for the other chains); fc_set_workspace registers a caller-owned DEVICE
 * buffer (256-byte aligned) for the current device, used by later fc_run calls until replaced.
 */
fc_status fc_workspace_size(const fc_chain_spec* spec, size_t* bytes);
fc_status fc_set_workspace(void* dev_ptr, size_t bytes);

/*
 * Collapsed form.  A 16-bit GEMM_NT whose ops are only BIAS_N, AFFINE_N and SCALE, reduced by ROW_SUM or
 * ROW_MEAN with store_main == 0, is not run as a GEMM: the sum over the output features commutes with
 * the contraction (the rewrite of the paper's showcase chain, linear layer -> sum over features),
 * out[m] = sum_k A[m][k] (sum_n a[n] B[n][k]) + sum_n c[n] with v -> a[n] v + c[n] the ops' effect, so
 * the weights and the activations are each read once.  Accumulated in fp64, rounded once to fp32.
 */

/*
 * Optional extra scratch.  A tensor-core chain (GEMM_NT or CONV2D_NHWC in bf16 / fp16) whose output
 * tiles do not fill the last round of SM pairs -- few rows, the regime of the paper's batch-sized
 * linear layers (appendix GEMM listing, which splits K and adds fp32 partials through a workspace), or
 * a ragged last round -- runs faster when those tiles are cut along K: the slices park fp32 partial
 * accumulators in scratch and the slice that finishes last adds them up in tensor memory and runs the
 * epilogue.  fc_workspace_size_split reports the workspace size that allows this for `spec`
 * (fc_workspace_size plus a fixed region of about 20 MB; 0 for chains that never split).  A smaller
 * workspace, or none where none is required, is not an error: fc_run then never splits.  Results are
 * the same up to fp32 summation order.
 * The size also covers one more optional use: a convolution with padding whose filter rows are short
 * (image layers of 8 to 32 channels: 5 x 5 x 8, 7 x 7 x 8, 3 x 3 x 16, 5 x 5 x 16) runs up to three times faster on a copy of the
 * image with its zero border written out, which fc_run makes in the workspace (one more kernel in front;
 * [batch][H + 2 pad][W + 2 pad][Cin] 16-bit elements, rounded up to 256 bytes, behind the channels-last copies
 * of CONV2D_NCHW) when the workspace has room for it and the problem is large enough for the extra launch to pay.  Results are the same up to fp32 summation order.
 */
fc_status fc_workspace_size_split(const fc_chain_spec* spec, size_t* bytes);

/*
 * Writes a one-line description of how fc_run would execute `spec` on the current device with the
 * workspace registered now: "kernel=ew_rowreduce", "kernel=gemm_f32", "kernel=collapse", "kernel=mlp_tc", or
 * "kernel=gemm_tc mode=<0 store|1 softmax|2 conv+pool|3 logsumexp> bn=<tile width> tiles=<256 x bn tiles>
 * pairs=<CTA pairs launched> split=<slices per split tile, 1 = none> split_tiles=<tiles that are split>
 * split_kb=<64-wide k-blocks per parking slice>" (a row softmax that takes its two-kernel form adds
 * " two_pass=1").  `text` is a caller-owned HOST buffer of `capacity`
 * bytes (truncated if too small).  Launches nothing.  For logs and tests; the format may gain fields.
 */
fc_status fc_describe_plan(const fc_chain_spec* spec, char* text, size_t capacity);

/*
 * GEMM_NT + ROW_SOFTMAX for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment convenience of this library.)
 *
 * Some callers have no allocator to hand: a plug-in that is given tensors but no memory pool, a
 * latency-critical loop or callback where cudaMalloc (which may synchronise the whole device) is
 * off limits, or a process whose device memory was reserved up front by another component.  They
 * cannot provide the workspace that fc_set_workspace wants.  This entry point runs the same kernel as fc_run, but takes its scratch
 * (per-tile row maxima and sums, per-panel arrival counters) from a fixed array that is part of
 * the library image: FC_STATIC_SCRATCH_BYTES bytes of device memory, resident on every GPU that
 * loads the library until the process exits.  The caller passes inputs and outputs exactly as to
 * fc_run (device pointers); nothing is allocated or freed, here or in any library this calls.
 *
 * Limits and rules.  Only GEMM_NT with reduce == FC_RED_ROW_SOFTMAX; other chains return
 * FC_ERR_UNSUPPORTED.  The scratch a call needs is
 *     2 * roundup(ceil(M / 128) * 4, 256)  +  M * ceil(N / 256) * 8   bytes
 * (arrival and departure counters per 128-row panel, then one (max, sum) pair per row and 256-column
 * tile).  That is about half of what fc_workspace_size reports for the same spec, because fc_run
 * reserves room for its two-kernel form as well; a spec that needs more than FC_STATIC_SCRATCH_BYTES
 * returns FC_ERR_WORKSPACE ("needs N bytes, the built-in scratch holds M").  Rows wider than 16384
 * columns (64 tiles), or with more tiles than CTA pairs are resident on the device, would need that
 * two-kernel form and return FC_ERR_UNSUPPORTED ("use fc_run").  All three checks come before the
 * device is touched.  The first call on each device
 * looks up the array's device address (with that device current); make that first call outside
 * any stream capture.  All calls on a device share the one array, which keeps whatever the last
 * call left in it: the counters are cleared on the stream before each launch, and two calls that
 * overlap on the GPU (different streams, no dependency) race on it and give wrong results.
 */
#define FC_STATIC_SCRATCH_BYTES (1u << 20)
fc_status fc_run_softmax_static_scratch(const fc_chain_spec* spec, const fc_tensor* inputs, int n_inputs,
                                        fc_tensor* outputs, int n_outputs, void* cuda_stream);

/*
 * Synchronises `cuda_stream`, then reads and clears the device status word of the current
 * device.  Returns FC_OK, FC_ERR_TIMEOUT (a bounded device-side wait expired in some launch since
 * the last call) or FC_ERR_CUDA.
 */
fc_status fc_get_async_status(void* cuda_stream);

/* Number of kernels this library has launched in this process (all devices, all threads). */
uint64_t fc_launch_count(void);

const char* fc_status_string(fc_status s);
const char* fc_last_error(void);   /* thread-local text of the last failure in this thread */
/* Thread-local, space-separated names of the kernel variants that the last fc_run of this thread enqueued ("ew_rows",
 * "ew_narrow", "gemm_tc_mode1_bn256_two_pass softmax_rescale", ...): which path a chain took, for logs and tests. */
const char* fc_last_plan(void);
int fc_version(void);

/*
 * Testing switches (process-wide, default 0; the paper has no counterpart).  FC_TESTING_PANEL_STALL / _SPLIT_STALL:
 * value 1 makes the named bounded wait expect one arrival too many (see "Testing aid" above).
 */
#define FC_TESTING_PANEL_STALL 0
#define FC_TESTING_SPLIT_STALL 1
#define FC_TESTING_BOUNDS_TRIP 2   /* debug build only: value 1 shortens the checked extent of the main output by one row */
#define FC_TESTING_TILE_WIDTH 3    /* value 128, 240 or 256: the column-tile width of every tensor-core GEMM that has a choice
                                      (plain store, row reductions, single-pass softmax, the fp32 form); 0: the launcher's own */
#define FC_TESTING_POOL_FORM 4     /* value 1, 2 or 3: the form of the 2x2 max-pool behind a convolution (1: every window through
                                      atomics; 2: windows inside a tile finished on chip; 3: tiles of whole row pairs, where the
                                      shape allows them, else the launcher's own); 0: the launcher's own */
#define FC_TESTING_BORDER_PASS 5   /* value 1: a few-channel convolution with padding runs on the bordered copy of its image
                                      whenever the workspace has room, whatever its size (0: from about eight rounds of tiles on) */
void fc_testing_set(int which, int value);

#ifdef __cplusplus
}
#endif
#endif /* FC_H_ */
