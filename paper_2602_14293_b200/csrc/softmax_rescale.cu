// Second pass of a GEMM + row softmax whose rows are wider than the tiles the SM pairs can hold at once.
//
// The single-pass kernel keeps every tile of a 256-row panel in tensor memory until the panel's last tile has
// published its (max, sum); that needs no more tiles per panel than the pairs have accumulator buffers (two
// each).  For wider rows (a vocabulary) the GEMM kernel does not wait: every tile stores its exponentials
// against the maximum of its half row (values in (0, 1]) and leaves (max_j, sum_j) per row, tile and column half in the
// workspace.
// This kernel gives a CTA to a row: it merges the row's pairs and rescales the stored values of half tile j by
// 2^((max_j - max_row) log2 e) / sum_row, in place.  HBM-bound: the probabilities are read and written once more.
#include "dev_common.cuh"

namespace fc {
namespace {

constexpr int kRescaleThreads = 256;

__global__ void __launch_bounds__(kRescaleThreads) softmax_rescale_kernel(void* out, int out_dt, const float2* __restrict__ stats,
                                                                          long long M, long long N, int tiles_n, int bn) {
    __shared__ MaxSum red[kRescaleThreads / 32];
    asm volatile("griddepcontrol.wait;" ::: "memory");   // launched programmatically behind the GEMM kernel
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool f16 = out_dt == FC_F16;
    for (long long m = blockIdx.x; m < M; m += gridDim.x) {
        const int halves = 2 * tiles_n, hw = bn >> 1;   // one pair per tile and column half
        const float2* st = stats + m * halves;
        MaxSum a = ms_identity();
        for (int j = threadIdx.x; j < halves; j += kRescaleThreads) {
            const float2 t = __ldcg(st + j);
            a = ms_merge(a, MaxSum{t.x, t.y});
        }
        a = ms_warp_reduce(a);
        __syncthreads();   // the previous row's readers are done with `red`
        if (lane == 0) red[warp] = a;
        __syncthreads();
        a = red[0];
#pragma unroll
        for (int w = 1; w < kRescaleThreads / 32; ++w) a = ms_merge(a, red[w]);
        const float inv = 1.0f / a.s;
        if (out_dt != FC_F32 && (N & 7) == 0 && (reinterpret_cast<uintptr_t>(out) & 15) == 0) {
            uint4* row = reinterpret_cast<uint4*>((unsigned short*) out + m * N);
            const int chunks = (int) (N >> 3), per_tile = hw >> 3;
            for (int c = threadIdx.x; c < chunks; c += kRescaleThreads) {
                const float mj = __ldcg(st + c / per_tile).x;
                const float f = mj == -CUDART_INF_F ? 0.0f : exp2_fast((mj - a.m) * kLog2e) * inv;
                const float2 f2 = make_float2(f, f);
                const uint4 q = row[c];
                const float2 x0 = __fmul2_rn(unpack16x2(q.x, f16), f2), x1 = __fmul2_rn(unpack16x2(q.y, f16), f2);
                const float2 x2 = __fmul2_rn(unpack16x2(q.z, f16), f2), x3 = __fmul2_rn(unpack16x2(q.w, f16), f2);
                uint4 o;
                o.x = pack16x2(x0.x, x0.y, f16); o.y = pack16x2(x1.x, x1.y, f16);
                o.z = pack16x2(x2.x, x2.y, f16); o.w = pack16x2(x3.x, x3.y, f16);
                row[c] = o;
            }
        } else {
            for (long long n = threadIdx.x; n < N; n += kRescaleThreads) {
                const float mj = __ldcg(st + n / hw).x;
                const float f = mj == -CUDART_INF_F ? 0.0f : exp2_fast((mj - a.m) * kLog2e) * inv;
                if (out_dt == FC_F32) {
                    float* o = (float*) out + m * N + n;
                    *o = *o * f;
                } else {
                    unsigned short* o = (unsigned short*) out + m * N + n;
                    const float x = unpack16x2((uint32_t) *o, f16).x * f;
                    *o = (unsigned short) (pack16x2(x, 0.0f, f16) & 0xffffu);
                }
            }
        }
    }
}

}  // namespace

cudaError_t launch_softmax_rescale(void* out, int out_dt, const float2* stats, long long M, long long N, int tiles_n, int bn,
                                   int num_sms, cudaStream_t stream, int* launches) {
    cudaLaunchConfig_t cfg = {};
    const long long want = (long long) num_sms * 8;
    cfg.gridDim = dim3((unsigned) (M < want ? M : want));
    cfg.blockDim = dim3(kRescaleThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    ++*launches;
    note_kernel("softmax_rescale");
    return cudaLaunchKernelEx(&cfg, softmax_rescale_kernel, out, out_dt, stats, M, N, tiles_n, bn);
}

}  // namespace fc
