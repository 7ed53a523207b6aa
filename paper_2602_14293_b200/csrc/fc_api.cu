// Host side of the C ABI: spec validation, kernel selection, TMA descriptor encoding, launch.
// Nothing here allocates device memory or synchronises (fc_get_async_status excepted).
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "fc_internal.h"

namespace fc {

__device__ int g_status_word;  // written by kernels when a bounded wait expires

namespace {

// testing switches (fc_testing_set): read on every call, written by tests only
std::atomic<int> g_inject_panel_stall{0}, g_inject_split_stall{0}, g_bounds_trip{0}, g_force_tile_width{0}, g_force_pool_form{0}, g_force_border_pass{0};

thread_local int t_device = 0;   // ordinal of the current device, noted by get_device at the top of every entry point
thread_local char t_err[512] = "";
thread_local char t_plan[256] = "";
std::atomic<uint64_t> g_launches{0};

fc_status fail(fc_status s, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(t_err, sizeof(t_err), fmt, ap);
    va_end(ap);
    return s;
}

constexpr int kMaxDevices = 64;
struct DeviceInfo {
    std::atomic<bool> ready{false};   // set last, with release: a reader that sees it sees the fields below
    int cc_major = 0, num_sms = 0;
    int* status = nullptr;
    void* workspace = nullptr;
    size_t workspace_bytes = 0;
    uint64_t counter_layout = 0;   // which counter layout the workspace was last left clean for (0: none)
};
DeviceInfo g_dev[kMaxDevices];
std::mutex g_mu;

// copy streams and events of fc_run_host's chunk pipeline, created on first use per device
struct HostPipe {
    static constexpr int kEvents = 2 + 2 * 8;
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev[kEvents] = {};
    std::mutex mu;
};
HostPipe g_pipe[kMaxDevices];

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode_tiled = nullptr;
EncodeIm2colFn g_encode_im2col = nullptr;

fc_status get_device(DeviceInfo** out, int* dev_out = nullptr) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(FC_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return fail(FC_ERR_CUDA, "device ordinal %d out of range", dev);
    DeviceInfo& d = g_dev[dev];
    t_device = dev;
    if (d.ready.load(std::memory_order_acquire)) {   // every call but the first on a device: no lock
        *out = &d;
        if (dev_out) *dev_out = dev;
        return FC_OK;
    }
    std::lock_guard<std::mutex> lk(g_mu);
    if (!d.ready.load(std::memory_order_relaxed)) {
        if ((e = cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return fail(FC_ERR_CUDA, "cudaDeviceGetAttribute: %s", cudaGetErrorString(e));
        if (d.cc_major != 10) return fail(FC_ERR_ARCH, "device %d has compute capability %d.x; sm_100a is required", dev, d.cc_major);
        if ((e = cudaGetSymbolAddress((void**) &d.status, g_status_word)) != cudaSuccess)
            return fail(FC_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        if (!g_encode_tiled) {
            cudaDriverEntryPointQueryResult q;
            void* fn = nullptr;
            e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
            if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn)
                return fail(FC_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
            g_encode_tiled = (EncodeTiledFn) fn;
            fn = nullptr;
            e = cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &fn, cudaEnableDefault, &q);
            if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn)
                return fail(FC_ERR_CUDA, "cuTensorMapEncodeIm2col entry point not available");
            g_encode_im2col = (EncodeIm2colFn) fn;
        }
        d.ready.store(true, std::memory_order_release);
    }
    *out = &d;
    if (dev_out) *dev_out = dev;
    return FC_OK;
}

size_t dt_size(int dt) { return dt == FC_F32 ? 4 : (dt == FC_F8E4M3 || dt == FC_E8M0 || dt == FC_MXF8E4M3 ? 1 : 2); }
bool dt_valid(int dt) { return dt == FC_F32 || dt == FC_BF16 || dt == FC_F16 || dt == FC_F8E4M3 || dt == FC_E8M0; }   // of a tensor (FC_MXF8E4M3 names a spec's operand format, not a tensor's)

// ------------------------------------------------------------------------------- validation
struct Plan {
    enum Kind { EW, GEMM_F32, TC_PLAIN, TC_SOFTMAX, TC_LSE, TC_CONV, GEMM_COLLAPSE, TC_MLP, TC_MX } kind;
    long long out_rows, out_cols;  // main output viewed as [rows][cols]
    int n_prod_inputs;
    int n_outputs;
    int main_index, red_index;     // indices into outputs[], -1 if absent
};

bool contiguous(const fc_tensor& t) {
    long long s = 1;
    for (int i = t.rank - 1; i >= 0; --i) {
        if (t.shape[i] != 1 && t.stride[i] != s) return false;
        s *= t.shape[i];
    }
    return true;
}

fc_status check_tensor(const fc_tensor& t, const char* what, int dtype_or_any, int rank, const long long* shape) {
    if (!t.ptr) return fail(FC_ERR_NULL, "%s: null pointer", what);
    if (!dt_valid(t.dtype)) return fail(FC_ERR_INVALID_SPEC, "%s: unknown dtype %d", what, t.dtype);
    if (dtype_or_any >= 0 && t.dtype != dtype_or_any) return fail(FC_ERR_INVALID_SPEC, "%s: dtype %d, expected %d", what, t.dtype, dtype_or_any);
    if (t.rank != rank) return fail(FC_ERR_SHAPE, "%s: rank %d, expected %d", what, t.rank, rank);
    for (int i = 0; i < rank; ++i)
        if (t.shape[i] != shape[i]) return fail(FC_ERR_SHAPE, "%s: shape[%d] = %lld, expected %lld", what, i, (long long) t.shape[i], shape[i]);
    if (!contiguous(t)) return fail(FC_ERR_UNSUPPORTED, "%s: only contiguous row-major tensors are supported", what);
    if (reinterpret_cast<uintptr_t>(t.ptr) % dt_size(t.dtype)) return fail(FC_ERR_ALIGNMENT, "%s: pointer not aligned to its element size", what);
    return FC_OK;
}

// MAXPOOL_2X2 stores its output as the spec's out_dtype when that is a 16-bit type (the next layer's operand type), else as fp32
bool pooled_16bit(const fc_chain_spec* s) { return s->reduce == FC_RED_MAXPOOL_2X2 && (s->out_dtype == FC_BF16 || s->out_dtype == FC_F16); }

bool is_conv(const fc_chain_spec* s) { return s->producer == FC_PROD_CONV2D_NHWC || s->producer == FC_PROD_CONV2D_NCHW; }

// CONV2D_NCHW: channels-last copies of the image and of the weights at the head of the workspace
size_t nchw_image_bytes(const fc_chain_spec* s) { return ((size_t) s->batch * s->H * s->W * s->Cin * 2 + 255) / 256 * 256; }
size_t nchw_workspace_bytes(const fc_chain_spec* s) {
    return nchw_image_bytes(s) + ((size_t) s->Cout * s->R * s->S * s->Cin * 2 + 255) / 256 * 256;
}

}  // namespace

void note_kernel(const char* name) {
    const size_t have = strlen(t_plan);
    snprintf(t_plan + have, sizeof(t_plan) - have, "%s%s", have ? " " : "", name);
}

namespace {

fc_status validate_spec(const fc_chain_spec* s, Plan* plan) {
    if (!s) return fail(FC_ERR_NULL, "spec is null");
    if (s->struct_size != sizeof(fc_chain_spec)) return fail(FC_ERR_INVALID_SPEC, "struct_size %u, expected %zu", s->struct_size, sizeof(fc_chain_spec));
    if (s->version != FC_VERSION) return fail(FC_ERR_INVALID_SPEC, "version %u, expected %d", s->version, FC_VERSION);
    if (s->producer < 0 || s->producer > FC_PROD_CONV2D_NCHW) return fail(FC_ERR_INVALID_SPEC, "unknown producer %d", s->producer);
    if ((!dt_valid(s->in_dtype) && s->in_dtype != FC_MXF8E4M3) || !dt_valid(s->out_dtype) || s->in_dtype == FC_E8M0)
        return fail(FC_ERR_INVALID_SPEC, "unknown in/out dtype");
    if (s->acc_dtype != FC_F32) return fail(FC_ERR_INVALID_SPEC, "acc_dtype must be FC_F32");
    if (s->out_dtype == FC_F8E4M3 || s->out_dtype == FC_E8M0) return fail(FC_ERR_UNSUPPORTED, "8-bit types are operand types only (outputs are fp32, bf16 or fp16)");
    if ((s->in_dtype == FC_F8E4M3 || s->in_dtype == FC_MXF8E4M3) && s->producer != FC_PROD_GEMM_NT) return fail(FC_ERR_UNSUPPORTED, "8-bit operands need a GEMM_NT producer");
    if (s->in_dtype == FC_MXF8E4M3 && s->reduce != FC_RED_NONE) return fail(FC_ERR_UNSUPPORTED, "block-scaled operands support reduce NONE");
    if (s->reduce < 0 || s->reduce > FC_RED_MAXPOOL_2X2) return fail(FC_ERR_INVALID_SPEC, "unknown reduce %d", s->reduce);
    if (s->n_ops < 0 || s->n_ops > FC_MAX_OPS) return fail(FC_ERR_INVALID_SPEC, "n_ops %d out of range", s->n_ops);
    for (int i = 0; i < s->n_ops; ++i)
        if (s->ops[i].kind < 0 || s->ops[i].kind > FC_OP_LINEAR) return fail(FC_ERR_INVALID_SPEC, "op %d: unknown kind %d", i, s->ops[i].kind);

    plan->n_prod_inputs = s->producer == FC_PROD_ELEMENTWISE ? 1 : (s->in_dtype == FC_MXF8E4M3 ? 4 : 2);
    if (is_conv(s)) {
        if (s->batch < 1 || s->H < 1 || s->W < 1 || s->Cin < 1 || s->Cout < 1 || s->R < 1 || s->S < 1 || s->stride < 1 || s->pad < 0)
            return fail(FC_ERR_SHAPE, "conv dimensions must be positive (pad >= 0)");
        const long long OH = (s->H + 2 * s->pad - s->R) / s->stride + 1, OW = (s->W + 2 * s->pad - s->S) / s->stride + 1;
        if (s->H + 2 * s->pad < s->R || s->W + 2 * s->pad < s->S) return fail(FC_ERR_SHAPE, "filter larger than the padded image");
        plan->out_rows = s->batch * OH * OW;
        plan->out_cols = s->Cout;
        if (plan->out_rows > 0x7fffffffLL || s->R * s->S * s->Cin > 0x7fffffffLL) return fail(FC_ERR_SHAPE, "conv too large");
    } else {
        if (s->M < 1 || s->N < 1 || (s->producer == FC_PROD_GEMM_NT && s->K < 1)) return fail(FC_ERR_SHAPE, "M, N, K must be >= 1");
        if (s->producer == FC_PROD_GEMM_NT && (s->M > 0x7fffffffLL || s->N > 0x7fffffffLL || s->K > 0x7fffffffLL))
            return fail(FC_ERR_SHAPE, "GEMM dimension exceeds 2^31-1");
        plan->out_rows = s->M;
        plan->out_cols = s->N;
    }

    // supported patterns
    if (s->reduce == FC_RED_NONE && !s->store_main) return fail(FC_ERR_INVALID_SPEC, "chain has no output (no reduction and store_main = 0)");
    plan->main_index = plan->red_index = -1;
    switch (s->producer) {
        case FC_PROD_ELEMENTWISE:
            if (s->reduce == FC_RED_GLOBAL_AVGPOOL || s->reduce == FC_RED_MAXPOOL_2X2)
                return fail(FC_ERR_UNSUPPORTED, "elementwise producer supports reduce NONE, ROW_LOGSUMEXP, ROW_SOFTMAX, ROW_SUM, ROW_MAX or ROW_MEAN");
            plan->kind = Plan::EW;
            break;
        case FC_PROD_GEMM_NT:
            if (s->in_dtype == FC_F32) {
                if (s->reduce != FC_RED_NONE || s->out_dtype != FC_F32)
                    return fail(FC_ERR_UNSUPPORTED, "fp32 GEMM supports fp32 output without reduction");
                if (s->N > 65535LL * 32) return fail(FC_ERR_SHAPE, "fp32 GEMM supports N <= %lld", 65535LL * 32);
                plan->kind = Plan::GEMM_F32;
            } else if (s->in_dtype == FC_MXF8E4M3) {
                plan->kind = Plan::TC_MX;
            } else if (s->reduce == FC_RED_NONE) {
                plan->kind = Plan::TC_PLAIN;
            } else if (s->reduce == FC_RED_ROW_SOFTMAX) {
                plan->kind = Plan::TC_SOFTMAX;
            } else if (s->reduce == FC_RED_ROW_LOGSUMEXP || s->reduce == FC_RED_ROW_SUM || s->reduce == FC_RED_ROW_MAX || s->reduce == FC_RED_ROW_MEAN) {
                plan->kind = Plan::TC_LSE;   // any reduction of a row to one value
                // A sum or mean over the output features of a purely linear epilogue, with no main output,
                // commutes with the contraction: out = A (sum_n a[n] B[n][:]) + sum_n c[n]  (collapse.cu)
                bool linear = (s->reduce == FC_RED_ROW_SUM || s->reduce == FC_RED_ROW_MEAN) && !s->store_main && s->in_dtype != FC_F8E4M3;
                for (int i = 0; i < s->n_ops && linear; ++i)
                    linear = s->ops[i].kind == FC_OP_BIAS_N || s->ops[i].kind == FC_OP_AFFINE_N || s->ops[i].kind == FC_OP_SCALE;
                if (linear) plan->kind = Plan::GEMM_COLLAPSE;
            } else {
                return fail(FC_ERR_UNSUPPORTED, "16-bit GEMM supports reduce NONE, ROW_SOFTMAX, ROW_LOGSUMEXP, ROW_SUM, ROW_MAX or ROW_MEAN");
            }
            break;
        default:
            if (s->in_dtype == FC_F32 || (s->reduce != FC_RED_GLOBAL_AVGPOOL && s->reduce != FC_RED_MAXPOOL_2X2) || s->store_main)
                return fail(FC_ERR_UNSUPPORTED, "conv supports bf16 / fp16 input with GLOBAL_AVGPOOL or MAXPOOL_2X2 and store_main = 0");
            if (s->reduce == FC_RED_MAXPOOL_2X2) {
                // the pooled maximum is taken with unsigned atomics on fp32 bit patterns over a zeroed output
                if (s->n_ops < 1 || s->ops[s->n_ops - 1].kind != FC_OP_RELU)
                    return fail(FC_ERR_UNSUPPORTED, "MAXPOOL_2X2 needs an op list that ends with RELU");
                const long long OH = (s->H + 2 * s->pad - s->R) / s->stride + 1, OW = (s->W + 2 * s->pad - s->S) / s->stride + 1;
                if (OH < 2 || OW < 2) return fail(FC_ERR_SHAPE, "MAXPOOL_2X2 needs a conv output of at least 2 x 2 (is %lld x %lld)", OH, OW);
                // a 16-bit pooled output is stored, not reached through atomics: every window must lie inside one tile
                if (pooled_16bit(s) && !(OH % 2 == 0 && 2 * OW <= 128))
                    return fail(FC_ERR_UNSUPPORTED, "MAXPOOL_2X2 with a 16-bit out_dtype needs an even number of conv output rows and at most 64 columns (is %lld x %lld); use FC_F32", OH, OW);
            }
            if (s->stride > 8) return fail(FC_ERR_UNSUPPORTED, "conv supports stride <= 8");
            if (s->pad >= s->R || s->pad >= s->S || s->R > 16 || s->S > 16) return fail(FC_ERR_UNSUPPORTED, "conv supports pad < R,S <= 16");
            plan->kind = Plan::TC_CONV;
            break;
    }
    {
        int linears = 0;
        for (int i = 0; i < s->n_ops; ++i) linears += s->ops[i].kind == FC_OP_LINEAR;
        if (linears > 0) {
            if (plan->kind != Plan::TC_PLAIN)
                return fail(FC_ERR_UNSUPPORTED, "LINEAR ops need a 16-bit GEMM_NT producer with reduce NONE");
            if (linears > 3) return fail(FC_ERR_UNSUPPORTED, "at most three LINEAR ops (four layers)");
            if (s->in_dtype == FC_F8E4M3) return fail(FC_ERR_UNSUPPORTED, "LINEAR ops need bf16 or fp16 operands");
            // per-layer limits that do not depend on the tensors; widths are checked with the tensors
            int vecs = 0;
            for (int i = 0; i < s->n_ops; ++i) {
                const int k = s->ops[i].kind;
                if (k == FC_OP_ADD_TENSOR) return fail(FC_ERR_UNSUPPORTED, "ADD_TENSOR cannot be combined with LINEAR ops");
                if (k == FC_OP_LINEAR) vecs = 0;
                vecs += k == FC_OP_BIAS_N ? 1 : (k == FC_OP_AFFINE_N ? 2 : 0);
                if (vecs > 3) return fail(FC_ERR_UNSUPPORTED, "at most 3 per-column vector operands per layer");
            }
            if (s->N > 256 || s->N % 8) return fail(FC_ERR_UNSUPPORTED, "with LINEAR ops every layer width must be a multiple of 8 and <= 256 (N = %lld)", (long long) s->N);
            plan->kind = Plan::TC_MLP;
        }
    }
    if (plan->kind == Plan::TC_PLAIN || plan->kind == Plan::TC_SOFTMAX || plan->kind == Plan::TC_LSE || plan->kind == Plan::TC_CONV || plan->kind == Plan::TC_MX) {
        int vecs = 0;
        for (int i = 0; i < s->n_ops; ++i) vecs += s->ops[i].kind == FC_OP_BIAS_N ? 1 : (s->ops[i].kind == FC_OP_AFFINE_N ? 2 : 0);
        if (vecs > 3) return fail(FC_ERR_UNSUPPORTED, "tensor-core chains support at most 3 per-column vector operands");
    }
    int n = 0;
    if (s->reduce == FC_RED_ROW_SOFTMAX) {
        plan->main_index = n++;
    } else {
        if (s->store_main) plan->main_index = n++;
        if (s->reduce != FC_RED_NONE) plan->red_index = n++;
    }
    plan->n_outputs = n;
    return FC_OK;
}

fc_status validate_tensors(const fc_chain_spec* s, const Plan& plan, const fc_tensor* in, int n_in, const fc_tensor* out, int n_out) {
    if (!in || !out) return fail(FC_ERR_NULL, "inputs / outputs array is null");
    if (n_in < plan.n_prod_inputs) return fail(FC_ERR_INVALID_SPEC, "producer needs %d inputs, got %d", plan.n_prod_inputs, n_in);
    if (n_out != plan.n_outputs) return fail(FC_ERR_INVALID_SPEC, "chain has %d outputs, got %d", plan.n_outputs, n_out);
    fc_status st;
    if (s->producer == FC_PROD_ELEMENTWISE) {
        const long long sh[2] = {s->M, s->N};
        if ((st = check_tensor(in[0], "inputs[0]", s->in_dtype, 2, sh))) return st;
    } else if (s->producer == FC_PROD_GEMM_NT) {
        const long long sa[2] = {s->M, s->K}, sb[2] = {s->N, s->K};
        const int operand_dt = s->in_dtype == FC_MXF8E4M3 ? FC_F8E4M3 : s->in_dtype;
        if ((st = check_tensor(in[0], "inputs[0] (A)", operand_dt, 2, sa))) return st;
        if ((st = check_tensor(in[1], "inputs[1] (B)", operand_dt, 2, sb))) return st;
        if (s->in_dtype == FC_MXF8E4M3) {
            if (s->K % 128) return fail(FC_ERR_ALIGNMENT, "block-scaled operands need K %% 128 == 0 (K = %lld)", (long long) s->K);
            const long long ssa[2] = {s->M, s->K / 32}, ssb[2] = {s->N, s->K / 32};
            if ((st = check_tensor(in[2], "inputs[2] (scales of A)", FC_E8M0, 2, ssa))) return st;
            if ((st = check_tensor(in[3], "inputs[3] (scales of B)", FC_E8M0, 2, ssb))) return st;
            if ((reinterpret_cast<uintptr_t>(in[0].ptr) | reinterpret_cast<uintptr_t>(in[1].ptr) | reinterpret_cast<uintptr_t>(in[2].ptr) |
                 reinterpret_cast<uintptr_t>(in[3].ptr)) & 15)
                return fail(FC_ERR_ALIGNMENT, "block-scaled operands and their scales must be 16-byte aligned");
        } else if (s->in_dtype != FC_F32) {
            const int kq = s->in_dtype == FC_F8E4M3 ? 16 : 8;   // a row of K elements must be a multiple of 16 bytes
            if (s->K % kq) return fail(FC_ERR_ALIGNMENT, "this GEMM needs K %% %d == 0 (K = %lld)", kq, (long long) s->K);
            if ((reinterpret_cast<uintptr_t>(in[0].ptr) | reinterpret_cast<uintptr_t>(in[1].ptr)) & 15)
                return fail(FC_ERR_ALIGNMENT, "bf16 GEMM operands must be 16-byte aligned");
        }
    } else {
        const bool cf = s->producer == FC_PROD_CONV2D_NCHW;
        const long long si[4] = {s->batch, cf ? s->Cin : s->H, cf ? s->H : s->W, cf ? s->W : s->Cin};
        const long long sw[4] = {s->Cout, cf ? s->Cin : s->R, cf ? s->R : s->S, cf ? s->S : s->Cin};
        if ((st = check_tensor(in[0], "inputs[0] (image)", s->in_dtype, 4, si))) return st;
        if ((st = check_tensor(in[1], "inputs[1] (weights)", s->in_dtype, 4, sw))) return st;
        if (s->Cin % 8) return fail(FC_ERR_ALIGNMENT, "conv needs Cin %% 8 == 0 (Cin = %lld)", (long long) s->Cin);
        if ((reinterpret_cast<uintptr_t>(in[0].ptr) | reinterpret_cast<uintptr_t>(in[1].ptr)) & 15)
            return fail(FC_ERR_ALIGNMENT, "conv operands must be 16-byte aligned");
    }
    long long cur_cols = plan.out_cols;   // width of a row at this point of the op list (LINEAR ops change it)
    for (int i = 0; i < s->n_ops; ++i) {
        const fc_op& op = s->ops[i];
        char what[64];
        if (op.kind == FC_OP_LINEAR) {
            if (op.in0 < plan.n_prod_inputs || op.in0 >= n_in) return fail(FC_ERR_INVALID_SPEC, "op %d: operand index %d out of range", i, op.in0);
            const fc_tensor& w = in[op.in0];
            snprintf(what, sizeof(what), "inputs[%d] (op %d weights)", op.in0, i);
            if (w.rank != 2 || w.shape[1] != cur_cols) return fail(FC_ERR_SHAPE, "%s: expected [N_next, %lld]", what, cur_cols);
            const long long sw[2] = {w.shape[0], cur_cols};
            if ((st = check_tensor(w, what, s->in_dtype, 2, sw))) return st;
            bool more = false;   // another LINEAR follows: this width is the next weight matrix's row length
            for (int j = i + 1; j < s->n_ops; ++j) more = more || s->ops[j].kind == FC_OP_LINEAR;
            if (w.shape[0] < 1 || w.shape[0] > 256 || (more && w.shape[0] % 8))
                return fail(FC_ERR_UNSUPPORTED, "%s: layer width %lld must be <= 256 and, unless it is the last, a multiple of 8", what, (long long) w.shape[0]);
            if (reinterpret_cast<uintptr_t>(w.ptr) & 15) return fail(FC_ERR_ALIGNMENT, "%s must be 16-byte aligned", what);
            cur_cols = w.shape[0];
            continue;
        }
        const long long vec[1] = {cur_cols};
        if (op.kind == FC_OP_BIAS_N || op.kind == FC_OP_AFFINE_N) {
            const int idx[2] = {op.in0, op.in1};
            for (int k = 0; k < (op.kind == FC_OP_AFFINE_N ? 2 : 1); ++k) {
                if (idx[k] < plan.n_prod_inputs || idx[k] >= n_in) return fail(FC_ERR_INVALID_SPEC, "op %d: operand index %d out of range", i, idx[k]);
                snprintf(what, sizeof(what), "inputs[%d] (op %d vector)", idx[k], i);
                if ((st = check_tensor(in[idx[k]], what, -1, 1, vec))) return st;
                if (in[idx[k]].dtype == FC_F8E4M3 || in[idx[k]].dtype == FC_E8M0) return fail(FC_ERR_UNSUPPORTED, "%s: 8-bit vectors are not supported", what);
            }
        } else if (op.kind == FC_OP_ADD_TENSOR) {
            if (op.in0 < plan.n_prod_inputs || op.in0 >= n_in) return fail(FC_ERR_INVALID_SPEC, "op %d: operand index %d out of range", i, op.in0);
            snprintf(what, sizeof(what), "inputs[%d] (op %d tensor)", op.in0, i);
            if (in[op.in0].dtype == FC_F8E4M3 || in[op.in0].dtype == FC_E8M0) return fail(FC_ERR_UNSUPPORTED, "%s: 8-bit tensors are not supported", what);
            if (is_conv(s)) {
                const long long OH = (s->H + 2 * s->pad - s->R) / s->stride + 1, OW = (s->W + 2 * s->pad - s->S) / s->stride + 1;
                const long long sh[4] = {s->batch, OH, OW, s->Cout};
                if ((st = check_tensor(in[op.in0], what, -1, 4, sh))) return st;
            } else {
                const long long sh[2] = {s->M, s->N};
                if ((st = check_tensor(in[op.in0], what, -1, 2, sh))) return st;
            }
        } else if (op.kind == FC_OP_CLAMP && !(op.f0 <= op.f1)) {
            return fail(FC_ERR_INVALID_SPEC, "op %d: clamp bounds lo > hi", i);
        }
    }
    if (plan.main_index >= 0) {
        if (is_conv(s)) {
            const long long OH = (s->H + 2 * s->pad - s->R) / s->stride + 1, OW = (s->W + 2 * s->pad - s->S) / s->stride + 1;
            const long long sh[4] = {s->batch, OH, OW, s->Cout};
            if ((st = check_tensor(out[plan.main_index], "main output", s->out_dtype, 4, sh))) return st;
        } else {
            const long long sh[2] = {s->M, cur_cols};
            if ((st = check_tensor(out[plan.main_index], "main output", s->out_dtype, 2, sh))) return st;
        }
    }
    if (plan.red_index >= 0) {
        if (s->reduce == FC_RED_MAXPOOL_2X2) {
            const long long OH = (s->H + 2 * s->pad - s->R) / s->stride + 1, OW = (s->W + 2 * s->pad - s->S) / s->stride + 1;
            const long long sh[4] = {s->batch, OH / 2, OW / 2, s->Cout};
            if ((st = check_tensor(out[plan.red_index], "pooled output", pooled_16bit(s) ? s->out_dtype : FC_F32, 4, sh))) return st;
        } else if (s->reduce != FC_RED_GLOBAL_AVGPOOL) {
            const long long sh[1] = {s->M};
            if ((st = check_tensor(out[plan.red_index], "row reduction output", FC_F32, 1, sh))) return st;
        } else {
            const long long sh[2] = {s->batch, s->Cout};
            if ((st = check_tensor(out[plan.red_index], "pooled output", FC_F32, 2, sh))) return st;
        }
    }
    return FC_OK;
}

// fused form of an op list: [scale]? [bias | affine]? [relu | gelu]? [scale]? [clamp]? [add tensor]?
void fused_from(const fc_op* ops, int n, const fc_tensor* in, FusedOps* out) {
    FusedOps& f = *out;
    memset(&f, 0, sizeof(f));
    f.scale = 1.0f;
    f.pre_scale = 1.0f;
    int i = 0;
    // a leading SCALE counts as the front one only when something that it cannot be merged with follows (a vector
    // or an activation); a lone SCALE, or one in front of a clamp or a residual, is the ordinary post-activation one
    if (n >= 2 && ops[0].kind == FC_OP_SCALE &&
        (ops[1].kind == FC_OP_BIAS_N || ops[1].kind == FC_OP_AFFINE_N || ops[1].kind == FC_OP_RELU || ops[1].kind == FC_OP_GELU_TANH))
        f.pre_scale = ops[i++].f0;
    if (i < n && (ops[i].kind == FC_OP_BIAS_N || ops[i].kind == FC_OP_AFFINE_N)) f.pre = ops[i++].kind == FC_OP_BIAS_N ? 1 : 2;
    if (i < n && (ops[i].kind == FC_OP_RELU || ops[i].kind == FC_OP_GELU_TANH)) f.act = ops[i++].kind == FC_OP_RELU ? 1 : 2;
    if (i < n && ops[i].kind == FC_OP_SCALE) f.scale = ops[i++].f0;
    if (i < n && ops[i].kind == FC_OP_CLAMP) { f.clamp = 1; f.lo = ops[i].f0; f.hi = ops[i].f1; ++i; }
    if (i < n && ops[i].kind == FC_OP_ADD_TENSOR) { f.res = 1; f.res_ptr = in[ops[i].in0].ptr; f.res_dt = in[ops[i].in0].dtype; ++i; }
    f.valid = i == n;
}

void build_ops(const fc_chain_spec* s, const fc_tensor* in, DevOps* d) {
    d->n = s->n_ops;
    for (int i = 0; i < s->n_ops; ++i) {
        const fc_op& op = s->ops[i];
        DevOp& o = d->op[i];
        o.kind = op.kind;
        o.f0 = op.f0;
        o.f1 = op.f1;
        o.p0 = o.p1 = nullptr;
        o.dt0 = o.dt1 = FC_F32;
        if (op.kind == FC_OP_BIAS_N || op.kind == FC_OP_AFFINE_N || op.kind == FC_OP_ADD_TENSOR) {
            o.p0 = in[op.in0].ptr;
            o.dt0 = in[op.in0].dtype;
        }
        if (op.kind == FC_OP_AFFINE_N) {
            o.p1 = in[op.in1].ptr;
            o.dt1 = in[op.in1].dtype;
        }
    }
    fused_from(s->ops, s->n_ops, in, &d->fused);
}

constexpr int kSoftmaxBN = 256;
constexpr int kSoftmaxOnePassTiles = 64;       // widest row (in tiles) that the single-pass softmax can take safely
// where the single pass is also the faster form (measured, see gemm_tile_width): rows of up to 16 tiles at any depth
// of the contraction, rows of up to 32 tiles from K = 2048 on
constexpr int kSoftmaxOnePassBestTiles = 16, kSoftmaxOnePassWideTiles = 32, kSoftmaxOnePassWideMinK = 2048;

// arrival counters and departure counters, one of each per 128-row panel
size_t panel_counter_bytes(long long M) {
    const long long panels = (M + 127) / 128;
    return ((size_t) panels * 4 + 255) / 256 * 256;
}

// Column-tile width of the GEMM kernels (modes 0, 1, 3, 7), and for the row softmax the choice between its two forms.
// Small GEMMs (modes 0 and 3, 256-wide tiles on at most half of the SM pairs) take 128-wide tiles where this
// cost model says so.  Such a call is one round of tiles, so its time is the critical tile's: main loop (of the
// merging slice, when tiles are cut along K) + epilogue + merge.  Measured, in microseconds: a k-block 0.33
// (256 wide) / 0.30 (128 wide; 24 instead of 32 KB), the epilogue 6 / 3, merging a split tile 8 / 4.4.
// 128 x 1024 x 1024: 13.7 -> 11.2; 256 x 4096 x 4096: 23.0 -> 20.1; 16 x 8192 x 8192 stays at 256 (37 against 45).
// Everything else is rounds of tiles whose main loops the tensor pipe bounds, so the time goes with
// rounds x tile width: 240-column tiles where that product is smaller (4096 x 4096: 288 tiles = 4 rounds x 240
// against 256 tiles = 4 rounds x 256 on 74 pairs).  `p` has its split scratch attached already.
int gemm_tile_width(TcParams& p, const fc_chain_spec* s, int num_sms) {
    if (p.mode == 1) {
        // Row softmax over more tiles per panel than the pairs' accumulator buffers can hold until the panel is
        // complete (two per pair; with a margin: 64 tiles = 16384 columns) cannot wait across tiles: a second,
        // memory-bound kernel finishes the rows.  The same two-kernel form is also chosen where it is faster: the
        // single pass writes every probability once, the two-kernel form writes, re-reads and re-writes it, but its
        // tiles run in the L2-friendly order and wait for nobody.  Measured (one pass / two kernels, us): 4096 x 4096 x
        // K: 37.8 / 40.0 at K = 64, 46.2 / 52.2 at 1024, 58.3 / 70.7 at 2048, 75.7 / 91.2 at 3072, 96 / 118 at 4096;
        // 4096 x 6144 x 4096 142 / 157; 8192 x 7168 x 4096 329 / 343; 4096 x 8192 x 2048 101 / 110, x 4096 185 / 183;
        // 8192 x 8192 x 512 150 / 124, x 1024 157 / 142, x 4096 376 / 371; beyond 8192 columns the two kernels win
        // (8192 x 16384 x 4096: 1208 / 838).
        const int tiles_n = (int) ((s->N + kSoftmaxBN - 1) / kSoftmaxBN);
        TcPlan tp;
        p.two_pass = false;
        // (never more tiles per panel than SM pairs take part, whatever the device offers)
        p.two_pass = plan_gemm_tc(p, kSoftmaxBN, num_sms, &tp) != cudaSuccess || tiles_n > kSoftmaxOnePassTiles || tiles_n > tp.pairs ||
                     tiles_n > kSoftmaxOnePassWideTiles || (tiles_n > kSoftmaxOnePassBestTiles && s->K < kSoftmaxOnePassWideMinK);
        if (p.two_pass) return kSoftmaxBN;
    } else if (p.mode != 0 && p.mode != 3 && p.mode != 7) {
        return 256;
    }
    // testing only (fc_testing_set): a given width for every call that could take it, so that the tests can run one
    // shape on all three tile widths
    const int forced = g_force_tile_width.load(std::memory_order_relaxed);
    if (forced == 128 || forced == 240 || forced == 256) {
        TcPlan tp;
        const long long tn = (s->N + forced - 1) / forced;
        if (p.mode != 1 || (plan_gemm_tc(p, forced, num_sms, &tp) == cudaSuccess && tn <= tp.pairs && tn <= kSoftmaxOnePassTiles)) return forced;
    }
    if (p.mode != 1 && s->N <= 128) return 128;
    const long long tiles = ((s->M + 255) / 256) * ((s->N + 255) / 256);
    if (2 * tiles <= num_sms / 2) {
        if (p.mode == 1) return kSoftmaxBN;
        auto cost = [&](int bn) -> double {
            TcPlan tp;
            if (plan_gemm_tc(p, bn, num_sms, &tp) != cudaSuccess) return 1e30;
            const bool cut = tp.split > 1;
            const int kb = cut ? tp.num_kb - tp.split_kb * (tp.split - 1) : tp.num_kb;
            return bn == 256 ? kb * 0.33 + 6.0 + (cut ? 8.0 : 0.0) : kb * 0.30 + 3.0 + (cut ? 4.4 : 0.0);
        };
        return cost(128) < cost(256) ? 128 : 256;
    }
    // k-blocks on the critical path x columns per tile
    auto rounds = [&](int bn) -> double {
        TcPlan tp;
        if (plan_gemm_tc(p, bn, num_sms, &tp) != cudaSuccess || tp.pairs <= 0) return 1e30;
        if (p.mode == 1 && (s->N + bn - 1) / bn > tp.pairs) return 1e30;
        double kb;
        if (tp.split > 1) kb = (double) ((tp.tiles - tp.split_tiles) / tp.pairs) * tp.num_kb + (tp.num_kb - tp.split_kb * (tp.split - 1)) + 24.0;
        else kb = (double) ((tp.tiles + tp.pairs - 1) / tp.pairs) * tp.num_kb;
        return kb * bn;
    };
    return rounds(240) < 0.98 * rounds(256) ? 240 : 256;
}

// fp32 GEMMs on the tensor cores (three tf32 products per fp32 product, see split_tf32_kernel): from this much work
// on, where it beats the register-tiled fp32 kernels (2048^3: 454 us there); K a multiple of 4 (16-byte rows for TMA).
// The split operands, [M, 3K] and [N, 3K] fp32, live in the workspace; without one the fp32 kernels run.
constexpr long long kTf32MinWork = 1LL << 29;   // M * N * K
bool tf32x3_eligible(const fc_chain_spec* s) {
    return s->K % 4 == 0 && s->K <= 0x7fffffffLL / 3 && s->M * s->N >= (kTf32MinWork + s->K - 1) / s->K && s->N >= 64 && s->M >= 64;
}
size_t tf32x3_a_bytes(const fc_chain_spec* s) { return ((size_t) s->M * 3 * s->K * 4 + 255) / 256 * 256; }
size_t tf32x3_workspace_bytes(const fc_chain_spec* s) { return tf32x3_a_bytes(s) + (size_t) s->N * 3 * s->K * 4; }

size_t softmax_workspace_bytes(long long M, long long N, bool per_half = false) {
    const long long tiles_n = (N + kSoftmaxBN - 1) / kSoftmaxBN;
    return 2 * panel_counter_bytes(M) + (size_t) M * tiles_n * sizeof(float2) * (per_half ? 2 : 1);
}
// fc_run's row softmax may take the two-kernel form, which keeps a pair per row, tile and column half
// ... and the other row reductions may run with 128-column tiles (twice the tiles): the same room
size_t reduction_workspace_bytes(bool /*softmax*/, long long M, long long N) { return softmax_workspace_bytes(M, N, true); }

// The part of the caller's workspace behind the row-reduction statistics serves split tiles; without it
// (no workspace, or a smaller one) the tensor-core kernels simply never split.
size_t split_workspace_offset(size_t reduction_bytes) { return (reduction_bytes + 255) / 256 * 256; }

void attach_split_scratch(const DeviceInfo* dev, size_t reduction_bytes, TcParams* p) {
    const size_t off = split_workspace_offset(reduction_bytes);
    if (!dev->workspace || dev->workspace_bytes < off + kTcSplitBytes) return;
    p->split_counters = (unsigned int*) ((char*) dev->workspace + off);
    p->split_ws = (float4*) ((char*) dev->workspace + off + kTcSplitCounterBytes);
}

// The kernels hand every counter back at zero, so the counters are cleared on the stream only when
// the workspace may hold something else where this launch keeps them: after fc_set_workspace, after a
// launch with another layout (different panel count, different place of the split counters), and after
// a launch that ended in a timeout.  `p` has its counter pointers set already.
cudaError_t clear_counters_if_needed(DeviceInfo* dev, const TcParams& p, size_t panel_bytes, cudaStream_t stream) {
    const uint64_t split_off = p.split_counters ? (uint64_t) ((char*) p.split_counters - (char*) dev->workspace) + 1 : 0;
    const uint64_t key = ((uint64_t) panel_bytes << 32) ^ split_off ^ (1ull << 63);
    std::lock_guard<std::mutex> lk(g_mu);
    if (dev->counter_layout == key) return cudaSuccess;
    cudaError_t e = cudaSuccess;
    if (panel_bytes && (e = cudaMemsetAsync(p.counters, 0, 2 * panel_bytes, stream)) != cudaSuccess) return e;
    if (p.split_counters && (e = cudaMemsetAsync(p.split_counters, 0, kTcSplitCounterBytes, stream)) != cudaSuccess) return e;
    dev->counter_layout = key;
    return cudaSuccess;
}

// Tensor maps depend only on (pointer, extents, box, dtype): a step that runs the same chain on the same
// buffers again finds them here instead of encoding them anew (a few of the microseconds of every call).
struct MapKey {
    const void* ptr;
    long long d[8];   // extents and the other parameters the encoding depends on
    bool operator==(const MapKey& o) const { return ptr == o.ptr && memcmp(d, o.d, sizeof(d)) == 0; }
};
struct MapCache {   // one per host thread: no lock on the per-call path
    static constexpr int kSlots = 16;
    MapKey key[kSlots];
    CUtensorMap map[kSlots];
    bool used[kSlots] = {};
    int next = 0;
    bool find(const MapKey& k, CUtensorMap* out) {
        for (int i = 0; i < kSlots; ++i)
            if (used[i] && key[i] == k) { *out = map[i]; return true; }
        return false;
    }
    void put(const MapKey& k, const CUtensorMap& m) {
        key[next] = k; map[next] = m; used[next] = true;
        next = (next + 1) % kSlots;
    }
};
thread_local MapCache g_maps;

fc_status encode_2d(CUtensorMap* tm, const void* ptr, long long rows, long long cols, int box_rows, int dt = FC_BF16) {
    const int dev = t_device;
    const MapKey mk = {ptr, {2, rows, cols, box_rows, dt, dev, 0, 0}};
    if (g_maps.find(mk, tm)) return FC_OK;
    const cuuint64_t esize = dt == FC_F8E4M3 ? 1 : (dt == FC_F32 ? 4 : 2);
    const cuuint64_t dims[2] = {(cuuint64_t) cols, (cuuint64_t) rows};
    const cuuint64_t strides[1] = {(cuuint64_t) cols * esize};
    const cuuint32_t box[2] = {(cuuint32_t) (128 / esize), (cuuint32_t) box_rows};   // 128-byte rows
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType tdt = dt == FC_F8E4M3 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                    : dt == FC_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                    : (dt == FC_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
    CUresult r = g_encode_tiled(tm, tdt, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(FC_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d (rows %lld cols %lld)", (int) r, rows, cols);
    g_maps.put(mk, *tm);
    return FC_OK;
}

// Scale tiles of the block-scaled GEMM: rows of 128 words (512 bytes), one row per (128-row tile, k-block)
fc_status encode_scale_tiles(CUtensorMap* tm, const void* ptr, long long tile_rows, int box_rows) {
    const int dev = t_device;
    const MapKey mk = {ptr, {7, tile_rows, dev, box_rows, 0, 0, 0, 0}};
    if (g_maps.find(mk, tm)) return FC_OK;
    const cuuint64_t dims[2] = {128, (cuuint64_t) tile_rows};
    const cuuint64_t strides[1] = {512};
    const cuuint32_t box[2] = {128, (cuuint32_t) box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode_tiled(tm, CU_TENSOR_MAP_DATA_TYPE_INT32, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(FC_ERR_CUDA, "cuTensorMapEncodeTiled (scale tiles) failed with CUresult %d", (int) r);
    g_maps.put(mk, *tm);
    return FC_OK;
}

// Eight channels (a first layer: RGB padded to 8) leave 56 of a k-block's 64 channels empty; packing eight taps
// into a k-block instead cuts a 5 x 5 filter from 25 k-blocks to 4.  The eight small copies of such a k-block
// cost about 1.9 us against 0.35 - 0.65 us for one 64-channel copy (measured), so from 16 channels on the
// one-tap k-blocks are as fast or faster.
// Few input channels without padding: in channels-last storage the S taps of one filter row are S * Cin contiguous
// elements per output position, so a tensor map whose "pixel" has S * Cin channels and whose pixels lie Cin
// elements apart (they overlap) fetches a whole filter row of 128 positions in one im2col copy of 128-byte rows; what
// the 64-element box asks for beyond S * Cin is out of range and arrives as zeros, so the weight columns that the B
// tile holds there (the next filter row's) meet zeros.  A k-block per filter row: 5 x 5 x 8 costs 5 k-blocks of one
// copy each instead of 4 of eight 16-byte-row copies (measured: 1.9 us per such k-block in the TMA unit).  Not with
// padding: a position whose first tap lies left of the image would lose its whole row, not just that tap.
// Longer filter rows (16 channels x 5 taps, 32 x 3) go in 64-element pieces, as long as that makes fewer k-blocks than a
// k-block per tap does (channel counts below 64 that do not divide it evenly into taps: 5 x 5 x 16 takes 10 instead of 25).
bool short_rows(const fc_chain_spec* s) {
    return s->Cin % 8 == 0 && s->Cin < 64 && s->S > 1 && s->S * s->Cin <= 256 && (s->S * s->Cin + 63) / 64 < s->S;
}
bool row_taps(const fc_chain_spec* s) { return short_rows(s) && s->pad == 0; }
// The same shapes with padding take that form too when the caller's workspace has room for a copy of the image with its
// zero border written out (a layout pass in front, as for channel-first operands: 85 MB for 4096 images of 32 x 32 x 8
// with a border of 2, written in about 25 us, against 1.9 us per k-block of eight small copies in the convolution).
// (the border pass is one more trip over the image: worth it against the eight small copies of an eight-channel
// k-block, 1.9 us each, and where the pieces are at most half as many as the taps: 3 x 3 x 32 on 256 images of 56 x 56,
// 6 k-blocks instead of 9, measured 143 against 146 us into 64 channels and 186 against 169 into 128)
bool padded_rows(const fc_chain_spec* s) {
    return short_rows(s) && s->pad > 0 && (s->Cin == 8 || 2 * ((s->S * s->Cin + 63) / 64) <= s->S);
}
size_t padded_image_bytes(const fc_chain_spec* s) {
    return ((size_t) s->batch * (s->H + 2 * s->pad) * (s->W + 2 * s->pad) * s->Cin * 2 + 255) / 256 * 256;
}
bool use_padded_rows(const fc_chain_spec* s, const DeviceInfo* dev) {
    // (channel-first operands: behind their channels-last copies)
    const size_t front = s->producer == FC_PROD_CONV2D_NCHW ? nchw_workspace_bytes(s) : 0;
    if (!padded_rows(s) || !dev->workspace || dev->workspace_bytes < front + padded_image_bytes(s)) return false;
    // The border pass is a launch of its own that the convolution waits for (about 6 us): it pays from some eight rounds
    // of tiles on (64 images of 32 x 32 x 8, 5 x 5, 3.5 rounds: 38.9 us either way; 8 images: 20.5 without, 22.5 with;
    // 4096 images: 1587 without, 743 with).  FC_TESTING_BORDER_PASS = 1 takes it at any size.
    if (g_force_border_pass.load(std::memory_order_relaxed)) return true;
    const long long OH = (s->H + 2 * s->pad - s->R) / s->stride + 1, OW = (s->W + 2 * s->pad - s->S) / s->stride + 1;
    const long long bn = s->Cout <= 64 ? 64 : (s->Cout <= 128 ? 128 : 256);
    const long long tiles = ((s->batch * OH * OW + 255) / 256) * ((s->Cout + bn - 1) / bn);
    return tiles >= 8LL * (dev->num_sms / 2);
}
// (the convolution that runs behind the border pass: the bordered image, no padding)
fc_chain_spec bordered_spec(const fc_chain_spec* s) {
    fc_chain_spec b = *s;
    b.H += 2 * s->pad;
    b.W += 2 * s->pad;
    b.pad = 0;
    return b;
}
bool packed_taps(const fc_chain_spec* s) { return s->Cin == 8 && !row_taps(s); }

// `packed`: copies of 8 channels x 128 pixels without swizzle (one column of 8 x 16-byte core matrices each), for
// channel counts that do not fill 64-channel k-blocks; otherwise 64 channels x 128 pixels with 128-byte swizzle.
fc_status encode_im2col(CUtensorMap* tm, const fc_chain_spec* s, const void* ptr, bool packed) {
    const int dev = t_device;
    const bool rows = !packed && row_taps(s);
    const MapKey mk = {ptr, {packed ? 5 : (rows ? 6 : 4), s->batch * 65536 + dev, s->H, s->W, s->Cin, s->R * 64 + s->S, s->stride * 64 + s->pad, s->in_dtype}};
    if (g_maps.find(mk, tm)) return FC_OK;
    // (row taps: a "pixel" of S * Cin channels; the pixel stride stays Cin elements)
    const cuuint64_t dims[4] = {(cuuint64_t) (rows ? s->S * s->Cin : s->Cin), (cuuint64_t) s->W, (cuuint64_t) s->H, (cuuint64_t) s->batch};
    const cuuint64_t strides[3] = {(cuuint64_t) s->Cin * 2, (cuuint64_t) s->W * s->Cin * 2, (cuuint64_t) s->H * s->W * s->Cin * 2};
    // base pixels run over the output grid shifted by -pad; a filter tap adds (s, r) to every base pixel
    const int lower[2] = {(int) -s->pad, (int) -s->pad};
    const int upper[2] = {(int) (s->pad - (s->S - 1)), (int) (s->pad - (s->R - 1))};
    // base pixels advance by the convolution stride along w and h
    const cuuint32_t estr[4] = {1, (cuuint32_t) s->stride, (cuuint32_t) s->stride, 1};
    CUresult r = g_encode_im2col(tm, s->in_dtype == FC_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, lower, upper,
                                 packed ? 8 : 64, 128, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, packed ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(FC_ERR_CUDA, "cuTensorMapEncodeIm2col failed with CUresult %d", (int) r);
    g_maps.put(mk, *tm);
    return FC_OK;
}

// The convolution's launch parameters that depend on the spec alone (fc_run adds pointers and the workspace).
int conv_params(const fc_chain_spec* spec, long long out_rows, TcParams* p) {
    p->mode = 2;
    p->batch = (int) spec->batch; p->H = (int) spec->H; p->W = (int) spec->W; p->Cin = (int) spec->Cin; p->Cout = (int) spec->Cout;
    p->R = (int) spec->R; p->S = (int) spec->S; p->stride = (int) spec->stride; p->pad = (int) spec->pad;
    p->OH = (int) ((spec->H + 2 * spec->pad - spec->R) / spec->stride + 1);
    p->OW = (int) ((spec->W + 2 * spec->pad - spec->S) / spec->stride + 1);
    p->M = (int) out_rows; p->N = (int) spec->Cout; p->K = (int) (spec->R * spec->S * spec->Cin);
    p->group_m = 1;
    p->in_dt = spec->in_dtype;
    p->inv_hw = 1.0f / (float) (p->OH * p->OW);
    // max-pool: 1 = every window through atomics, merged per warp; 2 = windows that lie inside a CTA's 128 consecutive
    // positions finished on chip and stored (78 % of them at OW = 28, 92 % at 10), the others through atomics.  The
    // second form costs two 128-thread barriers per channel chunk: from OW = 56 on it measured slower (105 -> 110 us).
    p->pool = spec->reduce == FC_RED_MAXPOOL_2X2 ? (p->OW <= 32 ? 2 : 1) : 0;
    // Tiles of whole row pairs: with an even number of output rows per image every image is a whole number of row pairs
    // (2 * OW consecutive positions), and a CTA whose tile stands for the largest number of whole pairs that fits its
    // 128 positions (112 of them at OW = 28 or 56, 120 at OW = 10) holds all four positions of every window it
    // touches: the second form then finishes every window on chip, no atomics are left, and the output needs no zeros
    // in front.  The price is the positions that a tile loads and multiplies but leaves to the next one (up to 12.5 %).
    p->m_rows = 128;
    p->pool_whole = 0;
    const int forced = g_force_pool_form.load(std::memory_order_relaxed);
    const bool whole_ok = p->pool && p->OH % 2 == 0 && 2 * p->OW <= 128;
    const bool must = pooled_16bit(spec);     // (validated: whole_ok holds)
    if (p->pool && forced >= 1 && forced <= 2 && !must) p->pool = forced;
    // fp32 outputs: where no position of a tile is wasted (2 * OW divides 128: 33.8 against 35.9 us on 64 images of
    // 32 x 32 x 64 -> 128), where the other choice is atomics for every window (OW > 32: F3 103.5 against 105.4 us), and
    // where a tile's few k-blocks leave the epilogue in the open (a 5 x 5 x 8 -> 64 image layer 640 against 664 us).
    // Elsewhere the up to 14 % more tiles cost more than the few atomics left (5 x 5 x 64 -> 128 at OW = 10: 208.9
    // against 203.6 us).  16-bit outputs always: they cannot be reached through atomics.
    const int kbs = row_taps(spec) ? (int) (spec->R * ((spec->S * spec->Cin + 63) / 64)) : (packed_taps(spec) ? (int) ((spec->R * spec->S * spec->Cin + 63) / 64) : (int) (spec->R * spec->S * ((spec->Cin + 63) / 64)));
    const bool pays = 128 % (2 * p->OW) == 0 || p->OW > 32 || kbs <= 8;
    if (whole_ok && (forced == 3 || (forced == 0 && pays) || must)) {
        p->pool = 2;
        p->pool_whole = 1;
        p->m_rows = 128 / (2 * p->OW) * (2 * p->OW);
    }
    p->a_packed = packed_taps(spec);
    p->a_rowtaps = row_taps(spec);
    // (up to 64 output channels: 64-column tiles, so that both column halves of the epilogue warps have work: with
    // 128-column tiles half of them idled and a 5 x 5 x 8 -> 64 layer, whose five k-blocks per tile the epilogue cannot
    // hide behind, was bound by the other half)
    const int bn = spec->Cout <= 64 ? 64 : (spec->Cout <= 128 ? 128 : 256);
    return bn;
}

fc_status cuda_fail(cudaError_t e, const char* what) { return fail(FC_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e)); }

}  // namespace
}  // namespace fc

using namespace fc;

extern "C" {

fc_status fc_run(const fc_chain_spec* spec, const fc_tensor* inputs, int n_inputs, fc_tensor* outputs, int n_outputs,
                 void* cuda_stream) {
    Plan plan;
    fc_status st;
    t_plan[0] = 0;
    if ((st = validate_spec(spec, &plan))) return st;
    if ((st = validate_tensors(spec, plan, inputs, n_inputs, outputs, n_outputs))) return st;
    DeviceInfo* dev;
    if ((st = get_device(&dev))) return st;
    cudaStream_t stream = (cudaStream_t) cuda_stream;
    int launches = 0;
    cudaError_t e = cudaSuccess;

    switch (plan.kind) {
        case Plan::EW: {
            EwParams p;
            p.status = dev->status;
            p.dbg_trim = g_bounds_trip.load(std::memory_order_relaxed) ? spec->N * (long long) dt_size(spec->out_dtype) : 0;
            p.x = inputs[0].ptr; p.x_dt = spec->in_dtype;
            p.y = plan.main_index >= 0 ? outputs[plan.main_index].ptr : nullptr;
            p.y_dt = spec->out_dtype;
            p.red = plan.red_index >= 0 ? (float*) outputs[plan.red_index].ptr : nullptr;
            p.M = spec->M; p.N = spec->N; p.reduce = spec->reduce;
            build_ops(spec, inputs, &p.ops);
            e = launch_ew_rowreduce(p, dev->num_sms, stream, &launches);
            break;
        }
        case Plan::GEMM_F32: {
            if (tf32x3_eligible(spec) && dev->workspace && dev->workspace_bytes >= tf32x3_workspace_bytes(spec) &&
                ((reinterpret_cast<uintptr_t>(inputs[0].ptr) | reinterpret_cast<uintptr_t>(inputs[1].ptr)) & 15) == 0) {
                {   // the split operands overwrite whatever counters a previous layout kept here
                    std::lock_guard<std::mutex> lk(g_mu);
                    dev->counter_layout = 0;
                }
                float* a3 = (float*) dev->workspace;
                float* b3 = (float*) ((char*) dev->workspace + tf32x3_a_bytes(spec));
                if ((e = launch_split_tf32((const float*) inputs[0].ptr, a3, spec->M, spec->K, false, false, stream, &launches)) != cudaSuccess) return cuda_fail(e, "operand split kernel launch");
                if ((e = launch_split_tf32((const float*) inputs[1].ptr, b3, spec->N, spec->K, true, true, stream, &launches)) != cudaSuccess) return cuda_fail(e, "operand split kernel launch");
                TcParams p;
                memset(&p, 0, sizeof(p));
                p.mode = 7;
                p.M = (int) spec->M; p.N = (int) spec->N; p.K = (int) (3 * spec->K);
                p.in_dt = FC_F32;
                p.out = outputs[plan.main_index].ptr; p.out_dt = FC_F32;
                p.status = dev->status;
                p.dbg_trim = g_bounds_trip.load(std::memory_order_relaxed) ? spec->N * 4LL : 0;
                build_ops(spec, inputs, &p.ops);
                {
                    const long long panel_bytes = 256LL * p.K * 4;
                    long long g = (32LL << 20) / (panel_bytes > 0 ? panel_bytes : 1);
                    p.group_m = (int) (g < 1 ? 1 : (g > 64 ? 64 : g));
                }
                const int bn = gemm_tile_width(p, spec, dev->num_sms);
                CUtensorMap tmA, tmB;
                if ((st = encode_2d(&tmA, a3, spec->M, p.K, 128, FC_F32))) return st;
                if ((st = encode_2d(&tmB, b3, spec->N, p.K, bn / 2, FC_F32))) return st;   // each CTA of a pair loads half
                e = launch_gemm_tc(p, tmA, tmB, bn, dev->num_sms, stream, &launches);
                break;
            }
            GemmF32Params p;
            p.A = (const float*) inputs[0].ptr; p.B = (const float*) inputs[1].ptr;
            p.C = (float*) outputs[plan.main_index].ptr;
            p.M = (int) spec->M; p.N = (int) spec->N; p.K = (int) spec->K;
            build_ops(spec, inputs, &p.ops);
            e = launch_gemm_f32(p, stream, &launches);
            break;
        }
        case Plan::TC_PLAIN:
        case Plan::TC_LSE:
        case Plan::TC_SOFTMAX: {
            TcParams p;
            memset(&p, 0, sizeof(p));
            p.mode = plan.kind == Plan::TC_SOFTMAX ? 1 : (plan.kind == Plan::TC_LSE ? 3 : 0);
            p.M = (int) spec->M; p.N = (int) spec->N; p.K = (int) spec->K;
            p.in_dt = spec->in_dtype;
            p.out = plan.main_index >= 0 ? outputs[plan.main_index].ptr : nullptr; p.out_dt = spec->out_dtype;
            p.red = plan.red_index >= 0 ? (float*) outputs[plan.red_index].ptr : nullptr;
            p.red_kind = spec->reduce;
            p.status = dev->status;
            p.dbg_trim = g_bounds_trip.load(std::memory_order_relaxed) ? spec->N * (long long) dt_size(spec->out_dtype) : 0;
            build_ops(spec, inputs, &p.ops);
            {
                // keep about 32 MB of A rows (group_m panels of 256 rows) resident in L2 per sweep
                const long long panel_bytes = 256LL * spec->K * (long long) dt_size(spec->in_dtype);
                long long g = (32LL << 20) / (panel_bytes > 0 ? panel_bytes : 1);
                p.group_m = (int) (g < 1 ? 1 : (g > 64 ? 64 : g));
            }
            // testing only (fc_testing_set): the panel wait, or the wait of a split tile's merging slice, expects one
            // arrival that never comes, so that the bounded wait expires and the call ends with FC_ERR_TIMEOUT
            p.expect_extra = (p.mode == 1 ? g_inject_panel_stall : g_inject_split_stall).load(std::memory_order_relaxed) ? 1 : 0;
            size_t panel_bytes = 0;
            if (p.mode == 1 || p.mode == 3) {
                const size_t need = reduction_workspace_bytes(p.mode == 1, spec->M, spec->N);
                if (!dev->workspace || dev->workspace_bytes < need)
                    return fail(FC_ERR_WORKSPACE, "this row reduction needs a %zu-byte workspace (fc_set_workspace); have %zu", need, dev->workspace_bytes);
                panel_bytes = panel_counter_bytes(spec->M);
                p.counters = (unsigned int*) dev->workspace;
                p.departed = (unsigned int*) ((char*) dev->workspace + panel_bytes);
                p.stats = (float2*) ((char*) dev->workspace + 2 * panel_bytes);
            }
            attach_split_scratch(dev, p.mode == 1 || p.mode == 3 ? reduction_workspace_bytes(p.mode == 1, spec->M, spec->N) : 0, &p);
            if ((e = clear_counters_if_needed(dev, p, panel_bytes, stream)) != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
            const int bn = gemm_tile_width(p, spec, dev->num_sms);   // (row softmax: also decides p.two_pass)
            CUtensorMap tmA, tmB;
            if ((st = encode_2d(&tmA, inputs[0].ptr, spec->M, spec->K, 128, spec->in_dtype))) return st;
            if ((st = encode_2d(&tmB, inputs[1].ptr, spec->N, spec->K, bn / 2, spec->in_dtype))) return st;   // each CTA of a pair loads half
            const int tiles_n = (int) ((spec->N + bn - 1) / bn);
            e = launch_gemm_tc(p, tmA, tmB, bn, dev->num_sms, stream, &launches);
            if (e == cudaSuccess && p.two_pass)
                e = launch_softmax_rescale(p.out, p.out_dt, p.stats, spec->M, spec->N, tiles_n, bn, dev->num_sms, stream, &launches);
            break;
        }
        case Plan::TC_MX: {
            const int bn = mx_tile_width(spec->N), parts = (bn + 127) / 128;
            const size_t sa_bytes = (scale_tiles_bytes(spec->M, spec->K, 128) + 255) / 256 * 256, sb_bytes = scale_tiles_bytes(spec->N, spec->K, bn);
            if (!dev->workspace || dev->workspace_bytes < sa_bytes + sb_bytes)
                return fail(FC_ERR_WORKSPACE, "block-scaled operands need a %zu-byte workspace (fc_set_workspace); have %zu", sa_bytes + sb_bytes, dev->workspace_bytes);
            {   // the scale tiles overwrite whatever counters a previous layout kept here
                std::lock_guard<std::mutex> lk(g_mu);
                dev->counter_layout = 0;
            }
            void* sa_tiles = dev->workspace;
            void* sb_tiles = (char*) dev->workspace + sa_bytes;
            if ((e = launch_scale_tiles(inputs[2].ptr, sa_tiles, spec->M, spec->K, 128, false, stream, &launches)) != cudaSuccess) return cuda_fail(e, "scale-tile kernel launch");
            if ((e = launch_scale_tiles(inputs[3].ptr, sb_tiles, spec->N, spec->K, bn, true, stream, &launches)) != cudaSuccess) return cuda_fail(e, "scale-tile kernel launch");
            TcParams p;
            memset(&p, 0, sizeof(p));
            p.mode = 6;
            p.M = (int) spec->M; p.N = (int) spec->N; p.K = (int) spec->K;
            p.in_dt = FC_F8E4M3;   // the elements; the scales come through their own tensor maps
            p.out = outputs[plan.main_index].ptr; p.out_dt = spec->out_dtype;
            p.status = dev->status;
            build_ops(spec, inputs, &p.ops);
            {
                const long long panel_bytes = 256LL * spec->K;
                long long g = (32LL << 20) / (panel_bytes > 0 ? panel_bytes : 1);
                p.group_m = (int) (g < 1 ? 1 : (g > 64 ? 64 : g));
            }
            CUtensorMap tmA, tmB, tmSA, tmSB;
            if ((st = encode_2d(&tmA, inputs[0].ptr, spec->M, spec->K, 128, FC_F8E4M3))) return st;
            if ((st = encode_2d(&tmB, inputs[1].ptr, spec->N, spec->K, bn / 2, FC_F8E4M3))) return st;   // each CTA of a pair loads half of the tile's rows of B
            if ((st = encode_scale_tiles(&tmSA, sa_tiles, (long long) ((spec->M + 127) / 128) * (spec->K / 128), 1))) return st;
            if ((st = encode_scale_tiles(&tmSB, sb_tiles, (long long) ((spec->N + bn - 1) / bn) * (spec->K / 128) * parts, parts))) return st;
            e = launch_gemm_tc_mx(p, tmA, tmB, tmSA, tmSB, dev->num_sms, stream, &launches);
            break;
        }
        case Plan::TC_MLP: {
            MlpParams p;
            memset(&p, 0, sizeof(p));
            p.M = (int) spec->M; p.K0 = (int) spec->K;
            p.in_dt = spec->in_dtype;
            p.out = outputs[plan.main_index].ptr; p.out_dt = spec->out_dtype;
            p.status = dev->status;
            p.width[0] = (int) spec->N;
            CUtensorMap tmX, tmW[4];
            auto box_rows = [](long long w) { return (int) ((w + 15) / 16 * 8); };   // each CTA of a pair loads half of the width padded to the MMA's N step
            if ((st = encode_2d(&tmX, inputs[0].ptr, spec->M, spec->K, 128, spec->in_dtype))) return st;
            if ((st = encode_2d(&tmW[0], inputs[1].ptr, spec->N, spec->K, box_rows(spec->N), spec->in_dtype))) return st;
            int l = 0;
            for (int i = 0; i < spec->n_ops; ++i) {
                const fc_op& op = spec->ops[i];
                if (op.kind == FC_OP_LINEAR) {
                    const fc_tensor& w = inputs[op.in0];
                    ++l;
                    p.width[l] = (int) w.shape[0];
                    if ((st = encode_2d(&tmW[l], w.ptr, w.shape[0], w.shape[1], box_rows(w.shape[0]), spec->in_dtype))) return st;
                    continue;
                }
                DevOps& d = p.seg[l];
                DevOp& o = d.op[d.n++];
                o.kind = op.kind; o.f0 = op.f0; o.f1 = op.f1;
                o.p0 = o.p1 = nullptr; o.dt0 = o.dt1 = FC_F32;
                if (op.kind == FC_OP_BIAS_N || op.kind == FC_OP_AFFINE_N) { o.p0 = inputs[op.in0].ptr; o.dt0 = inputs[op.in0].dtype; }
                if (op.kind == FC_OP_AFFINE_N) { o.p1 = inputs[op.in1].ptr; o.dt1 = inputs[op.in1].dtype; }
            }
            p.layers = l + 1;
            {
                // the packed straight-line form of each layer's ops, where the list has the usual shape
                int first = 0;
                for (int seg = 0, i = 0; i <= spec->n_ops; ++i) {
                    if (i == spec->n_ops || spec->ops[i].kind == FC_OP_LINEAR) {
                        fused_from(spec->ops + first, i - first, inputs, &p.seg[seg].fused);
                        first = i + 1;
                        ++seg;
                    }
                }
            }
            e = launch_mlp_tc(p, tmX, tmW, dev->num_sms, stream, &launches);
            break;
        }
        case Plan::GEMM_COLLAPSE: {
            const size_t need = collapse_workspace_bytes(spec->N, spec->K);
            if (!dev->workspace || dev->workspace_bytes < need)
                return fail(FC_ERR_WORKSPACE, "this chain needs a %zu-byte workspace (fc_set_workspace); have %zu", need, dev->workspace_bytes);
            {
                std::lock_guard<std::mutex> lk(g_mu);
                dev->counter_layout = 0;   // the collapsed weights overwrite where other chains keep counters
            }
            CollapseParams p;
            p.A = inputs[0].ptr; p.B = inputs[1].ptr; p.in_dt = spec->in_dtype;
            p.M = spec->M; p.N = spec->N; p.K = spec->K;
            build_ops(spec, inputs, &p.ops);
            p.out = (float*) outputs[plan.red_index].ptr;
            p.post = spec->reduce == FC_RED_ROW_MEAN ? 1.0f / (float) spec->N : 1.0f;
            e = launch_collapse(p, dev->workspace, dev->num_sms, stream, &launches);
            break;
        }
        case Plan::TC_CONV: {
            TcParams p;
            memset(&p, 0, sizeof(p));
            // (few channels with padding: the convolution runs without padding on a bordered copy of the image)
            const bool bordered = use_padded_rows(spec, dev);
            const fc_chain_spec border_spec = bordered ? bordered_spec(spec) : *spec;
            const fc_chain_spec* const user_spec = spec;
            if (bordered) spec = &border_spec;
            const int bn = conv_params(spec, plan.out_rows, &p);
            p.out = outputs[plan.red_index].ptr; p.out_dt = pooled_16bit(spec) ? spec->out_dtype : FC_F32;
            p.status = dev->status;
            build_ops(spec, inputs, &p.ops);
            const size_t out_elems = p.pool ? (size_t) spec->batch * (p.OH / 2) * (p.OW / 2) * spec->Cout : (size_t) spec->batch * spec->Cout;
            const void* image = inputs[0].ptr;
            const void* weights = inputs[1].ptr;
            size_t head = 0;   // workspace bytes in front of the split scratch
            if (user_spec->producer == FC_PROD_CONV2D_NCHW) {
                head = nchw_workspace_bytes(user_spec);
                if (!dev->workspace || dev->workspace_bytes < head)
                    return fail(FC_ERR_WORKSPACE, "CONV2D_NCHW needs a workspace of %zu bytes (fc_workspace_size)", head);
                void* img_cl = dev->workspace;
                void* w_cl = (char*) dev->workspace + nchw_image_bytes(user_spec);
                {   // the copies overwrite whatever counters a previous layout kept here
                    std::lock_guard<std::mutex> lk(g_mu);
                    dev->counter_layout = 0;
                }
                if ((e = launch_cfirst_to_clast(weights, w_cl, user_spec->Cout, p.Cin, p.R * p.S, false, stream, &launches)) != cudaSuccess)
                    return cuda_fail(e, "layout kernel launch");
                if ((e = launch_cfirst_to_clast(image, img_cl, user_spec->batch, p.Cin, (int) (user_spec->H * user_spec->W), true, stream, &launches)) != cudaSuccess)
                    return cuda_fail(e, "layout kernel launch");
                image = img_cl;
                weights = w_cl;
            }
            if (bordered) {
                // (behind the channels-last copies of channel-first operands, if any)
                void* img_b = (char*) dev->workspace + head;
                head += padded_image_bytes(user_spec);
                {   // the copy overwrites whatever counters a previous layout kept here
                    std::lock_guard<std::mutex> lk(g_mu);
                    dev->counter_layout = 0;
                }
                if ((e = launch_pad_image(image, img_b, user_spec->batch, (int) user_spec->H, (int) user_spec->W, (int) user_spec->Cin,
                                          (int) user_spec->pad, dev->num_sms, stream, &launches)) != cudaSuccess)
                    return cuda_fail(e, "border kernel launch");
                image = img_b;
            }
            attach_split_scratch(dev, head, &p);
            if ((e = clear_counters_if_needed(dev, p, 0, stream)) != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
            CUtensorMap tmA, tmB;
            if ((st = encode_im2col(&tmA, spec, image, p.a_packed != 0))) return st;
            if ((st = encode_2d(&tmB, weights, spec->Cout, p.K, bn / 2, spec->in_dtype))) return st;
            // The pooled output is cleared by a kernel directly in front of the convolution, which is launched
            // programmatically behind it: its loads and MMAs start at once, only its epilogue warps wait for the zeros.
            // (not for a max-pool over tiles of whole row pairs: every window is stored once, by the tile that holds it)
            if (!p.pool_whole) {
                if ((e = launch_zero_fill(p.out, out_elems * 4, dev->num_sms, stream, &launches)) != cudaSuccess) return cuda_fail(e, "zero-fill launch");
                p.after_zero_fill = 1;
            }
            e = launch_gemm_tc(p, tmA, tmB, bn, dev->num_sms, stream, &launches);
            break;
        }
    }
    g_launches.fetch_add((uint64_t) launches);
    if (e != cudaSuccess) return cuda_fail(e, "kernel launch");
    return FC_OK;
}

fc_status fc_staging_size(const fc_chain_spec* spec, const fc_tensor* inputs, int n_inputs, const fc_tensor* outputs,
                          int n_outputs, size_t* bytes) {
    if (!bytes || !inputs || !outputs) return fail(FC_ERR_NULL, "null argument");
    (void) spec;
    size_t total = 0;
    auto add = [&](const fc_tensor& t) {
        size_t n = dt_size(t.dtype);
        for (int i = 0; i < t.rank; ++i) n *= (size_t) t.shape[i];
        total += (n + 255) / 256 * 256;
    };
    for (int i = 0; i < n_inputs; ++i) add(inputs[i]);
    for (int i = 0; i < n_outputs; ++i) add(outputs[i]);
    *bytes = total;
    return FC_OK;
}

fc_status fc_run_host(const fc_chain_spec* spec, const fc_tensor* host_inputs, int n_inputs, fc_tensor* host_outputs,
                      int n_outputs, void* staging, size_t staging_bytes, void* cuda_stream) {
    Plan plan;
    fc_status st;
    if ((st = validate_spec(spec, &plan))) return st;
    if (!host_inputs || !host_outputs || !staging) return fail(FC_ERR_NULL, "null argument");
    if (n_inputs < 0 || n_inputs > 16 || n_outputs < 0 || n_outputs > 4) return fail(FC_ERR_INVALID_SPEC, "too many tensors");
    size_t need = 0;
    if ((st = fc_staging_size(spec, host_inputs, n_inputs, host_outputs, n_outputs, &need))) return st;
    if (staging_bytes < need) return fail(FC_ERR_WORKSPACE, "staging buffer has %zu bytes, %zu needed", staging_bytes, need);
    if (reinterpret_cast<uintptr_t>(staging) & 255) return fail(FC_ERR_ALIGNMENT, "staging buffer must be 256-byte aligned");
    cudaStream_t stream = (cudaStream_t) cuda_stream;
    fc_tensor din[16], dout[4];
    size_t nbytes_in[16], nbytes_out[4];
    char* cur = (char*) staging;
    size_t moved = 0;
    for (int i = 0; i < n_inputs; ++i) {
        if (!host_inputs[i].ptr) return fail(FC_ERR_NULL, "host_inputs[%d]: null pointer", i);
        size_t n = dt_size(host_inputs[i].dtype);
        for (int k = 0; k < host_inputs[i].rank; ++k) n *= (size_t) host_inputs[i].shape[k];
        nbytes_in[i] = n;
        din[i] = host_inputs[i];
        din[i].ptr = cur;
        cur += (n + 255) / 256 * 256;
        moved += n;
    }
    for (int i = 0; i < n_outputs; ++i) {
        if (!host_outputs[i].ptr) return fail(FC_ERR_NULL, "host_outputs[%d]: null pointer", i);
        size_t n = dt_size(host_outputs[i].dtype);
        for (int k = 0; k < host_outputs[i].rank; ++k) n *= (size_t) host_outputs[i].shape[k];
        nbytes_out[i] = n;
        dout[i] = host_outputs[i];
        dout[i].ptr = cur;
        cur += (n + 255) / 256 * 256;
        moved += n;
    }

    // Rows (images) are independent problems: large chains are cut into row chunks so that the
    // host-to-device copy of chunk i+1, the kernel of chunk i and the device-to-host copy of chunk
    // i-1 overlap (two internal copy streams; the kernels stay on the caller's stream).
    const bool conv = is_conv(spec);
    const long long rows = conv ? spec->batch : spec->M;
    const long long gran = (plan.kind == Plan::TC_PLAIN || plan.kind == Plan::TC_SOFTMAX || plan.kind == Plan::TC_LSE || plan.kind == Plan::TC_MLP) ? 256 : 1;
    long long chunks = 1;
    if (moved >= ((size_t) 32 << 20) && plan.kind != Plan::GEMM_F32 && plan.kind != Plan::GEMM_COLLAPSE && plan.kind != Plan::TC_MX && n_inputs >= plan.n_prod_inputs && n_outputs == plan.n_outputs) {
        chunks = rows / gran < 8 ? rows / gran : 8;
        if (chunks < 1) chunks = 1;
    }
    if (chunks == 1) {
        for (int i = 0; i < n_inputs; ++i) {
            cudaError_t e = cudaMemcpyAsync(din[i].ptr, host_inputs[i].ptr, nbytes_in[i], cudaMemcpyHostToDevice, stream);
            if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync H2D");
        }
        if ((st = fc_run(spec, din, n_inputs, dout, n_outputs, cuda_stream))) return st;
        for (int i = 0; i < n_outputs; ++i) {
            cudaError_t e = cudaMemcpyAsync(host_outputs[i].ptr, dout[i].ptr, nbytes_out[i], cudaMemcpyDeviceToHost, stream);
            if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync D2H");
        }
        return FC_OK;
    }

    // whole-shape validation first: the chunks below are validated against sub-shapes only
    if ((st = validate_tensors(spec, plan, din, n_inputs, dout, n_outputs))) return st;
    int ordinal = 0;
    DeviceInfo* dev;
    if ((st = get_device(&dev, &ordinal))) return st;
    HostPipe& hp = g_pipe[ordinal];
    std::lock_guard<std::mutex> lk(hp.mu);
    cudaError_t e;
    if (!hp.ready) {
        if ((e = cudaStreamCreateWithFlags(&hp.s_in, cudaStreamNonBlocking)) != cudaSuccess ||
            (e = cudaStreamCreateWithFlags(&hp.s_out, cudaStreamNonBlocking)) != cudaSuccess)
            return cuda_fail(e, "cudaStreamCreateWithFlags");
        for (int i = 0; i < HostPipe::kEvents; ++i)
            if ((e = cudaEventCreateWithFlags(&hp.ev[i], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e, "cudaEventCreateWithFlags");
        hp.ready = true;
    }
    bool split[16];
    for (int i = 0; i < n_inputs; ++i) split[i] = i == 0;
    for (int i = 0; i < spec->n_ops; ++i)
        if (spec->ops[i].kind == FC_OP_ADD_TENSOR) split[spec->ops[i].in0] = true;
    cudaEvent_t ev_start = hp.ev[0], ev_done = hp.ev[1];
#define FC_TRY(call, what) do { if ((e = (call)) != cudaSuccess) return cuda_fail(e, what); } while (0)
    FC_TRY(cudaEventRecord(ev_start, stream), "cudaEventRecord");
    FC_TRY(cudaStreamWaitEvent(hp.s_in, ev_start, 0), "cudaStreamWaitEvent");
    FC_TRY(cudaStreamWaitEvent(hp.s_out, ev_start, 0), "cudaStreamWaitEvent");
    for (int i = 0; i < n_inputs; ++i)
        if (!split[i]) FC_TRY(cudaMemcpyAsync(din[i].ptr, host_inputs[i].ptr, nbytes_in[i], cudaMemcpyHostToDevice, hp.s_in), "cudaMemcpyAsync H2D");
    const long long per = ((rows + chunks - 1) / chunks + gran - 1) / gran * gran;
    int c = 0;
    for (long long r0 = 0; r0 < rows; r0 += per, ++c) {
        const long long r1 = r0 + per < rows ? r0 + per : rows;
        fc_chain_spec sub = *spec;
        if (conv) sub.batch = r1 - r0; else sub.M = r1 - r0;
        fc_tensor sin[16], sout[4];
        for (int i = 0; i < n_inputs; ++i) {
            sin[i] = din[i];
            if (!split[i]) continue;
            const size_t row_bytes = nbytes_in[i] / (size_t) rows;
            sin[i].ptr = (char*) din[i].ptr + (size_t) r0 * row_bytes;
            sin[i].shape[0] = r1 - r0;
            FC_TRY(cudaMemcpyAsync(sin[i].ptr, (const char*) host_inputs[i].ptr + (size_t) r0 * row_bytes, (size_t) (r1 - r0) * row_bytes,
                                   cudaMemcpyHostToDevice, hp.s_in), "cudaMemcpyAsync H2D");
        }
        cudaEvent_t ev_in = hp.ev[2 + 2 * c], ev_k = hp.ev[3 + 2 * c];
        FC_TRY(cudaEventRecord(ev_in, hp.s_in), "cudaEventRecord");
        FC_TRY(cudaStreamWaitEvent(stream, ev_in, 0), "cudaStreamWaitEvent");
        for (int i = 0; i < n_outputs; ++i) {
            const size_t row_bytes = nbytes_out[i] / (size_t) rows;
            sout[i] = dout[i];
            sout[i].ptr = (char*) dout[i].ptr + (size_t) r0 * row_bytes;
            sout[i].shape[0] = r1 - r0;
        }
        if ((st = fc_run(&sub, sin, n_inputs, sout, n_outputs, cuda_stream))) return st;
        FC_TRY(cudaEventRecord(ev_k, stream), "cudaEventRecord");
        FC_TRY(cudaStreamWaitEvent(hp.s_out, ev_k, 0), "cudaStreamWaitEvent");
        for (int i = 0; i < n_outputs; ++i) {
            const size_t row_bytes = nbytes_out[i] / (size_t) rows;
            FC_TRY(cudaMemcpyAsync((char*) host_outputs[i].ptr + (size_t) r0 * row_bytes, sout[i].ptr, (size_t) (r1 - r0) * row_bytes,
                                   cudaMemcpyDeviceToHost, hp.s_out), "cudaMemcpyAsync D2H");
        }
    }
    FC_TRY(cudaEventRecord(ev_done, hp.s_out), "cudaEventRecord");
    FC_TRY(cudaStreamWaitEvent(stream, ev_done, 0), "cudaStreamWaitEvent");
#undef FC_TRY
    return FC_OK;
}

fc_status fc_workspace_size(const fc_chain_spec* spec, size_t* bytes) {
    Plan plan;
    fc_status st;
    if (!bytes) return fail(FC_ERR_NULL, "bytes is null");
    if ((st = validate_spec(spec, &plan))) return st;
    *bytes = plan.kind == Plan::TC_SOFTMAX || plan.kind == Plan::TC_LSE ? reduction_workspace_bytes(plan.kind == Plan::TC_SOFTMAX, spec->M, spec->N)
           : plan.kind == Plan::GEMM_COLLAPSE ? collapse_workspace_bytes(spec->N, spec->K)
           : plan.kind == Plan::GEMM_F32 ? (tf32x3_eligible(spec) ? tf32x3_workspace_bytes(spec) : 0)
           : plan.kind == Plan::TC_MX ? (spec->K % 128 ? 0 : (scale_tiles_bytes(spec->M, spec->K, 128) + 255) / 256 * 256 + scale_tiles_bytes(spec->N, spec->K, mx_tile_width(spec->N)))
           : spec->producer == FC_PROD_CONV2D_NCHW ? nchw_workspace_bytes(spec) : 0;
    return FC_OK;
}

fc_status fc_workspace_size_split(const fc_chain_spec* spec, size_t* bytes) {
    Plan plan;
    fc_status st;
    if (!bytes) return fail(FC_ERR_NULL, "bytes is null");
    if ((st = validate_spec(spec, &plan))) return st;
    const bool tc = plan.kind == Plan::TC_PLAIN || plan.kind == Plan::TC_SOFTMAX || plan.kind == Plan::TC_LSE || plan.kind == Plan::TC_CONV;
    const size_t red = plan.kind == Plan::TC_SOFTMAX || plan.kind == Plan::TC_LSE ? reduction_workspace_bytes(plan.kind == Plan::TC_SOFTMAX, spec->M, spec->N)
                     : plan.kind == Plan::TC_CONV ? (spec->producer == FC_PROD_CONV2D_NCHW ? nchw_workspace_bytes(spec) : 0) +
                                                     (padded_rows(spec) ? padded_image_bytes(spec) : 0)   // (the bordered copy of the image)
                     : 0;
    *bytes = tc ? split_workspace_offset(red) + kTcSplitBytes : 0;
    return FC_OK;
}

fc_status fc_describe_plan(const fc_chain_spec* spec, char* text, size_t capacity) {
    Plan plan;
    fc_status st;
    if (!text || capacity == 0) return fail(FC_ERR_NULL, "text is null or has no room");
    if ((st = validate_spec(spec, &plan))) return st;
    if (plan.kind == Plan::EW) { snprintf(text, capacity, "kernel=ew_rowreduce"); return FC_OK; }
    if (plan.kind == Plan::GEMM_F32) {
        DeviceInfo* d2;
        if ((st = get_device(&d2))) return st;
        const bool tf = tf32x3_eligible(spec) && d2->workspace && d2->workspace_bytes >= tf32x3_workspace_bytes(spec);
        snprintf(text, capacity, tf ? "kernel=gemm_tc mode=7" : "kernel=gemm_f32");
        return FC_OK;
    }
    if (plan.kind == Plan::GEMM_COLLAPSE) { snprintf(text, capacity, "kernel=collapse"); return FC_OK; }
    if (plan.kind == Plan::TC_MLP) { snprintf(text, capacity, "kernel=mlp_tc"); return FC_OK; }
    if (plan.kind == Plan::TC_MX) { snprintf(text, capacity, "kernel=gemm_tc mode=6 bn=%d", mx_tile_width(spec->N)); return FC_OK; }
    DeviceInfo* dev;
    if ((st = get_device(&dev))) return st;
    TcParams p;
    memset(&p, 0, sizeof(p));
    int bn;
    size_t red = 0;
    fc_chain_spec border_spec;
    if (plan.kind == Plan::TC_CONV) {
        if (spec->producer == FC_PROD_CONV2D_NCHW) red = nchw_workspace_bytes(spec);
        if (use_padded_rows(spec, dev)) {
            red += padded_image_bytes(spec);
            border_spec = bordered_spec(spec);
            spec = &border_spec;
        }
        bn = conv_params(spec, plan.out_rows, &p);
    } else {
        p.mode = plan.kind == Plan::TC_SOFTMAX ? 1 : (plan.kind == Plan::TC_LSE ? 3 : 0);
        p.M = (int) spec->M; p.N = (int) spec->N; p.K = (int) spec->K;
        p.in_dt = spec->in_dtype;
        bn = 0;
        if (p.mode == 1 || p.mode == 3) red = reduction_workspace_bytes(p.mode == 1, spec->M, spec->N);
    }
    attach_split_scratch(dev, red, &p);
    if (!bn) bn = gemm_tile_width(p, spec, dev->num_sms);
    TcPlan tp;
    cudaError_t e = plan_gemm_tc(p, bn, dev->num_sms, &tp);
    if (e != cudaSuccess) return cuda_fail(e, "planning");
    snprintf(text, capacity, "kernel=gemm_tc mode=%d bn=%d tiles=%d pairs=%d split=%d split_tiles=%d split_kb=%d%s", p.mode, tp.bn,
             tp.tiles, tp.pairs, tp.split, tp.split_tiles, tp.split_kb, p.mode == 1 && p.two_pass ? " two_pass=1" : "");
    return FC_OK;
}

fc_status fc_set_workspace(void* dev_ptr, size_t bytes) {
    if (dev_ptr && (reinterpret_cast<uintptr_t>(dev_ptr) & 255)) return fail(FC_ERR_ALIGNMENT, "workspace must be 256-byte aligned");
    DeviceInfo* dev;
    fc_status st;
    if ((st = get_device(&dev))) return st;
    std::lock_guard<std::mutex> lk(g_mu);
    dev->workspace = dev_ptr;
    dev->workspace_bytes = dev_ptr ? bytes : 0;
    dev->counter_layout = 0;
    return FC_OK;
}

fc_status fc_get_async_status(void* cuda_stream) {
    DeviceInfo* dev;
    fc_status st;
    if ((st = get_device(&dev))) return st;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t) cuda_stream);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    int word = 0;
    if ((e = cudaMemcpy(&word, dev->status, sizeof(int), cudaMemcpyDeviceToHost)) != cudaSuccess) return cuda_fail(e, "cudaMemcpy status");
    if (word != 0) {
        {
            std::lock_guard<std::mutex> lk(g_mu);
            dev->counter_layout = 0;   // the launch that gave up may have left counters behind
        }
        const int zero = 0;
        if ((e = cudaMemcpy(dev->status, &zero, sizeof(int), cudaMemcpyHostToDevice)) != cudaSuccess) return cuda_fail(e, "cudaMemcpy status");
        if ((word & 0xff) == FC_ERR_BOUNDS)   // debug build: the site of the first failed address check rides in the upper bits
            return fail(FC_ERR_BOUNDS, "a kernel computed an address outside one of its tensors (check site %d); the access was skipped", word >> 8);
        return fail((fc_status) word, "a bounded device-side wait expired");
    }
    return FC_OK;
}

uint64_t fc_launch_count(void) { return g_launches.load(); }

const char* fc_status_string(fc_status s) {
    switch (s) {
        case FC_OK: return "FC_OK";
        case FC_ERR_NULL: return "FC_ERR_NULL";
        case FC_ERR_INVALID_SPEC: return "FC_ERR_INVALID_SPEC";
        case FC_ERR_UNSUPPORTED: return "FC_ERR_UNSUPPORTED";
        case FC_ERR_SHAPE: return "FC_ERR_SHAPE";
        case FC_ERR_ALIGNMENT: return "FC_ERR_ALIGNMENT";
        case FC_ERR_WORKSPACE: return "FC_ERR_WORKSPACE";
        case FC_ERR_ARCH: return "FC_ERR_ARCH";
        case FC_ERR_CUDA: return "FC_ERR_CUDA";
        case FC_ERR_TIMEOUT: return "FC_ERR_TIMEOUT";
        case FC_ERR_BOUNDS: return "FC_ERR_BOUNDS";
    }
    return "FC_ERR_?";
}

const char* fc_last_error(void) { return t_err; }
const char* fc_last_plan(void) { return t_plan; }

int fc_version(void) { return FC_VERSION; }

void fc_testing_set(int which, int value) {
    if (which == FC_TESTING_PANEL_STALL) g_inject_panel_stall.store(value);
    else if (which == FC_TESTING_SPLIT_STALL) g_inject_split_stall.store(value);
    else if (which == FC_TESTING_BOUNDS_TRIP) g_bounds_trip.store(value);
    else if (which == FC_TESTING_TILE_WIDTH) g_force_tile_width.store(value);
    else if (which == FC_TESTING_POOL_FORM) g_force_pool_form.store(value);
    else if (which == FC_TESTING_BORDER_PASS) g_force_border_pass.store(value);
}

}  // extern "C"

// ------------------------------------------------------------------ built-in scratch (no allocation)
// Scratch of fc_run_softmax_static_scratch.  Lives in the library image on every device that loads
// it.  In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[FC_STATIC_SCRATCH_BYTES];

namespace {
void* g_static_scratch_ptr[fc::kMaxDevices] = {nullptr};   // device address per device, looked up once
}

extern "C" fc_status fc_run_softmax_static_scratch(const fc_chain_spec* spec, const fc_tensor* inputs, int n_inputs,
                                                   fc_tensor* outputs, int n_outputs, void* cuda_stream) {
    Plan plan;
    fc_status st;
    t_plan[0] = 0;
    if ((st = validate_spec(spec, &plan))) return st;
    if (plan.kind != Plan::TC_SOFTMAX) return fail(FC_ERR_UNSUPPORTED, "the built-in scratch serves GEMM_NT + ROW_SOFTMAX chains only");
    if ((st = validate_tensors(spec, plan, inputs, n_inputs, outputs, n_outputs))) return st;
    // size rules first, before anything touches the device
    const int tiles_n = (int) ((spec->N + kSoftmaxBN - 1) / kSoftmaxBN);
    if (tiles_n > kSoftmaxOnePassTiles)
        return fail(FC_ERR_UNSUPPORTED, "rows wider than %d columns take two kernels: use fc_run", kSoftmaxOnePassTiles * kSoftmaxBN);
    const size_t need = softmax_workspace_bytes(spec->M, spec->N);
    if (need > FC_STATIC_SCRATCH_BYTES)
        return fail(FC_ERR_WORKSPACE, "this chain needs %zu bytes of scratch, the built-in scratch holds %u", need, (unsigned) FC_STATIC_SCRATCH_BYTES);
    DeviceInfo* dev;
    int ordinal = 0;
    if ((st = get_device(&dev, &ordinal))) return st;
    void* scratch = nullptr;
    {
        // set-up, once per device, with that device current: the array's address on THIS device
        std::lock_guard<std::mutex> lk(g_mu);
        if (!g_static_scratch_ptr[ordinal]) {
            void* ptr = nullptr;
            cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
            if (e != cudaSuccess || !ptr) return fail(FC_ERR_CUDA, "cudaGetSymbolAddress(built-in scratch): %s", cudaGetErrorString(e));
            g_static_scratch_ptr[ordinal] = ptr;
        }
        scratch = g_static_scratch_ptr[ordinal];
    }
    cudaStream_t stream = (cudaStream_t) cuda_stream;
    TcParams p;
    memset(&p, 0, sizeof(p));
    p.mode = 1;
    p.M = (int) spec->M; p.N = (int) spec->N; p.K = (int) spec->K;
    p.out = outputs[plan.main_index].ptr; p.out_dt = spec->out_dtype;
    p.status = dev->status;
    build_ops(spec, inputs, &p.ops);
    const size_t counters = panel_counter_bytes(spec->M);
    p.group_m = 1;
    p.in_dt = spec->in_dtype;
    p.counters = (unsigned int*) scratch;
    p.departed = (unsigned int*) ((char*) scratch + counters);
    p.stats = (float2*) ((char*) scratch + 2 * counters);
    cudaError_t e;
    {
        // the same guard as fc_run: every tile of a row panel must be resident at once, so a panel may not have
        // more tiles than CTA pairs take part on this device (fewer SMs, a partitioned context)
        TcPlan tp;
        if ((e = plan_gemm_tc(p, kSoftmaxBN, dev->num_sms, &tp)) != cudaSuccess) return cuda_fail(e, "planning");
        if (tiles_n > tp.pairs)
            return fail(FC_ERR_UNSUPPORTED, "a row panel has %d tiles but only %d CTA pairs are resident on this device: use fc_run", tiles_n, tp.pairs);
    }
    // the array keeps the previous call's contents: the arrival and departure counters must start at zero
    if ((e = cudaMemsetAsync(p.counters, 0, 2 * counters, stream)) != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
    CUtensorMap tmA, tmB;
    if ((st = encode_2d(&tmA, inputs[0].ptr, spec->M, spec->K, 128, spec->in_dtype))) return st;
    if ((st = encode_2d(&tmB, inputs[1].ptr, spec->N, spec->K, kSoftmaxBN / 2, spec->in_dtype))) return st;
    int launches = 0;
    e = launch_gemm_tc(p, tmA, tmB, kSoftmaxBN, dev->num_sms, stream, &launches);
    g_launches.fetch_add((uint64_t) launches);
    if (e != cudaSuccess) return cuda_fail(e, "kernel launch");
    return FC_OK;
}
