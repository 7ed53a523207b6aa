// Kernel (a): memory-bound elementwise chain with an optional row logsumexp, one pass over the data.
//
// One CTA walks whole rows.  Each thread owns 16-byte chunks (8 bf16 or 4 fp32 values) at a fixed
// column stride, issues all its loads for a row (input and residual tensors) before any arithmetic,
// applies the op list in registers, stores the result once, and folds the fp32 values (before the
// output rounding) into a running (max, sum) pair.  Pairs are merged with warp shuffles and one
// shared-memory exchange per row.
//
// Two instantiations: a generic one (any op list, any N, any alignment) and a specialised one for
// "affine -> tanh-GELU -> add tensor -> logsumexp" on bf16 with the per-column vectors held in
// registers across rows.
#include "dev_common.cuh"

namespace fc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ MaxSum block_merge(MaxSum a, MaxSum* smem /* [kWarps] */) {
    a = ms_warp_reduce(a);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();  // smem reuse across rows
    if (lane == 0) smem[warp] = a;
    __syncthreads();
    MaxSum r = lane < kWarps ? smem[lane] : ms_identity();
    return ms_warp_reduce(r);
}

// ------------------------------------------------------------------------------------ generic
// Handles any dtype mix and tails with scalar access when 16-byte vectors are not possible.
template <bool kPreciseGelu>
__global__ void __launch_bounds__(kThreads) ew_generic_kernel(const EwParams p) {
    __shared__ MaxSum red[kWarps];
    const long long N = p.N;
    const int ebytes = p.x_dt == FC_BF16 ? 2 : 4;
    const int ybytes = p.y_dt == FC_BF16 ? 2 : 4;
    constexpr int kV = 8;  // columns per chunk
    const bool x_vec = ((reinterpret_cast<uintptr_t>(p.x) | (uintptr_t)(N * ebytes)) & 15) == 0;
    const bool y_vec = p.y && ((reinterpret_cast<uintptr_t>(p.y) | (uintptr_t)(N * ybytes)) & 15) == 0;
    const long long chunks = (N + kV - 1) / kV;

    for (long long m = blockIdx.x; m < p.M; m += gridDim.x) {
        MaxSum acc = ms_identity();
        for (long long c = threadIdx.x; c < chunks; c += kThreads) {
            const long long n0 = c * kV;
            const bool full = n0 + kV <= N;
            float v[kV];
            if (p.x_dt == FC_BF16) {
                if (full && x_vec) {
                    const uint4 q = __ldg(reinterpret_cast<const uint4*>((const unsigned short*) p.x + m * N + n0));
                    v[0] = bf16_lo(q.x); v[1] = bf16_hi(q.x); v[2] = bf16_lo(q.y); v[3] = bf16_hi(q.y);
                    v[4] = bf16_lo(q.z); v[5] = bf16_hi(q.z); v[6] = bf16_lo(q.w); v[7] = bf16_hi(q.w);
                } else {
#pragma unroll
                    for (int j = 0; j < kV; ++j) v[j] = n0 + j < N ? load_scalar(p.x, FC_BF16, m * N + n0 + j) : 0.0f;
                }
            } else {
                if (full && x_vec) {
                    const float4 a = __ldg(reinterpret_cast<const float4*>((const float*) p.x + m * N + n0));
                    const float4 b = __ldg(reinterpret_cast<const float4*>((const float*) p.x + m * N + n0 + 4));
                    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
                } else {
#pragma unroll
                    for (int j = 0; j < kV; ++j) v[j] = n0 + j < N ? load_scalar(p.x, FC_F32, m * N + n0 + j) : 0.0f;
                }
            }
            apply_ops<kV, kPreciseGelu>(v, p.ops, m, n0, N, N);
            if (p.reduce == FC_RED_ROW_LOGSUMEXP) {
                float mx = -CUDART_INF_F;
#pragma unroll
                for (int j = 0; j < kV; ++j) mx = n0 + j < N ? fmaxf(mx, v[j]) : mx;
                float s = 0.0f;
#pragma unroll
                for (int j = 0; j < kV; ++j) s += n0 + j < N ? exp2_fast((v[j] - mx) * kLog2e) : 0.0f;
                acc = ms_merge(acc, MaxSum{mx, s});
            }
            if (p.y) {
                if (p.y_dt == FC_BF16) {
                    unsigned short* yp = (unsigned short*) p.y + m * N + n0;
                    if (full && y_vec) {
                        uint4 q;
                        q.x = pack_bf16x2(v[0], v[1]); q.y = pack_bf16x2(v[2], v[3]);
                        q.z = pack_bf16x2(v[4], v[5]); q.w = pack_bf16x2(v[6], v[7]);
                        *reinterpret_cast<uint4*>(yp) = q;
                    } else {
#pragma unroll
                        for (int j = 0; j < kV; ++j)
                            if (n0 + j < N) yp[j] = (unsigned short) (pack_bf16x2(v[j], 0.0f) & 0xffffu);
                    }
                } else {
                    float* yp = (float*) p.y + m * N + n0;
                    if (full && y_vec) {
                        *reinterpret_cast<float4*>(yp) = make_float4(v[0], v[1], v[2], v[3]);
                        *reinterpret_cast<float4*>(yp + 4) = make_float4(v[4], v[5], v[6], v[7]);
                    } else {
#pragma unroll
                        for (int j = 0; j < kV; ++j)
                            if (n0 + j < N) yp[j] = v[j];
                    }
                }
            }
        }
        if (p.reduce == FC_RED_ROW_LOGSUMEXP) {
            const MaxSum t = block_merge(acc, red);
            if (threadIdx.x == 0) p.red[m] = t.m + logf(t.s);
        }
    }
}

}  // namespace

cudaError_t launch_ew_rowreduce(const EwParams& p, int num_sms, cudaStream_t stream, int* launches) {
    // precise GELU whenever an fp32 result (the logsumexp, or an fp32 main output) depends on it
    const bool precise = p.reduce == FC_RED_ROW_LOGSUMEXP || p.y_dt == FC_F32;
    long long grid = p.M < (long long) num_sms * 8 ? p.M : (long long) num_sms * 8;
    if (grid < 1) grid = 1;
    if (precise)
        ew_generic_kernel<true><<<(unsigned) grid, kThreads, 0, stream>>>(p);
    else
        ew_generic_kernel<false><<<(unsigned) grid, kThreads, 0, stream>>>(p);
    *launches += 1;
    return cudaGetLastError();
}

}  // namespace fc
