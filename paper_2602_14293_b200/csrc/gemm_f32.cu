// Strict-fp32 GEMM NT (C = epilogue(A * B^T), A [M,K], B [N,K], all fp32) for small problems.
//
// fp32 FMA on the plain ALUs: a single-pass TF32 tensor-core product would miss the fp32 output
// tolerance, and at the sizes this path serves (hundreds per side) the run time is launch latency.
// 32x32 output tile per CTA, 256 threads x (2x2) outputs, K staged through shared memory in
// slabs of 32 with register prefetch of the next slab.
#include "dev_common.cuh"

namespace fc {
namespace {

constexpr int kTile = 32;
constexpr int kSlab = 32;

__global__ void __launch_bounds__(256) gemm_f32_kernel(const GemmF32Params p) {
    __shared__ float As[kTile][kSlab + 1];
    __shared__ float Bs[kTile][kSlab + 1];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * kTile, n0 = blockIdx.x * kTile;
    // loader mapping: each thread moves 4 consecutive k of one row for A and for B
    const int lr = tid >> 3, lk = (tid & 7) * 4;
    const bool vec = ((reinterpret_cast<uintptr_t>(p.A) | reinterpret_cast<uintptr_t>(p.B)) & 15) == 0 && (p.K & 3) == 0;

    auto load4 = [&](const float* base, int row, int row_limit, int k) -> float4 {
        float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row < row_limit) {
            const float* q = base + (long long) row * p.K + k;
            if (vec && k + 3 < p.K) {
                r = __ldg(reinterpret_cast<const float4*>(q));
            } else {
                if (k + 0 < p.K) r.x = __ldg(q + 0);
                if (k + 1 < p.K) r.y = __ldg(q + 1);
                if (k + 2 < p.K) r.z = __ldg(q + 2);
                if (k + 3 < p.K) r.w = __ldg(q + 3);
            }
        }
        return r;
    };

    float acc[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
    float4 ra = load4(p.A, m0 + lr, p.M, lk);
    float4 rb = load4(p.B, n0 + lr, p.N, lk);
    for (int k0 = 0; k0 < p.K; k0 += kSlab) {
        As[lr][lk + 0] = ra.x; As[lr][lk + 1] = ra.y; As[lr][lk + 2] = ra.z; As[lr][lk + 3] = ra.w;
        Bs[lr][lk + 0] = rb.x; Bs[lr][lk + 1] = rb.y; Bs[lr][lk + 2] = rb.z; Bs[lr][lk + 3] = rb.w;
        __syncthreads();
        if (k0 + kSlab < p.K) {
            ra = load4(p.A, m0 + lr, p.M, k0 + kSlab + lk);
            rb = load4(p.B, n0 + lr, p.N, k0 + kSlab + lk);
        }
#pragma unroll
        for (int k = 0; k < kSlab; ++k) {
            const float a0 = As[ty * 2][k], a1 = As[ty * 2 + 1][k];
            const float b0 = Bs[tx * 2][k], b1 = Bs[tx * 2 + 1][k];
            acc[0][0] = fmaf(a0, b0, acc[0][0]);
            acc[0][1] = fmaf(a0, b1, acc[0][1]);
            acc[1][0] = fmaf(a1, b0, acc[1][0]);
            acc[1][1] = fmaf(a1, b1, acc[1][1]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int m = m0 + ty * 2 + i;
        if (m >= p.M) continue;
        float v[2] = {acc[i][0], acc[i][1]};
        const int n = n0 + tx * 2;
        apply_ops<2, false>(v, p.ops, m, n, p.N, p.N);
        if (n < p.N) p.C[(long long) m * p.N + n] = v[0];
        if (n + 1 < p.N) p.C[(long long) m * p.N + n + 1] = v[1];
    }
}

}  // namespace

cudaError_t launch_gemm_f32(const GemmF32Params& p, cudaStream_t stream, int* launches) {
    dim3 grid((p.N + kTile - 1) / kTile, (p.M + kTile - 1) / kTile);
    gemm_f32_kernel<<<grid, 256, 0, stream>>>(p);
    *launches += 1;
    return cudaGetLastError();
}

}  // namespace fc
