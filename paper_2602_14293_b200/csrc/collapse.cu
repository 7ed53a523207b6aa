// Linear layer followed by a row sum (or mean) with nothing non-linear in between: the reduction
// commutes with the contraction,
//
//     sum_n ( a[n] * sum_k A[m][k] B[n][k] + c[n] )  =  sum_k A[m][k] * u[k]  +  C,
//     u[k] = sum_n a[n] B[n][k],   C = sum_n c[n],
//
// where (a[n], c[n]) is what the chain's bias / affine / scale ops make of v -> a[n] v + c[n].  This is
// the algebraic rewrite of the paper's showcase chain (linear -> sum over the output features -> ...):
// the M x N x K contraction becomes one pass over the weights and one over the activations, both
// bound by HBM.  Three kernels, no atomics (results are reproducible bit for bit):
//
//   weight_colsum_kernel   partial[s][k] = sum over row slab s of a[n] B[n][k]; a warp adds 8 rows at a
//                          time in fp32 and the groups in fp64; block column 0 also sums c[n].
//   colsum_finish_kernel   u[k] = (float) sum_s partial[s][k],  C = sum_s cpart[s]   (fp64 sums)
//   row_dot_kernel         out[m] = post * (sum_k A[m][k] u[k] + C), a block per row or per 4 rows, each
//                          thread keeping its columns of u in registers; 8 products at a time in fp32,
//                          the groups in fp64, one rounding to fp32 at the end.
//
// Every fp32 rounding touches a partial sum of at most 8 terms (plus one rounding of u), so the result
// carries a relative error of about 1e-7 of the typical |out| whatever N and K are; converting every
// element to fp64 instead made the weight pass 30 % slower (conversions run at a quarter of the fp64
// FMA rate).
#include "dev_common.cuh"

namespace fc {
namespace {

constexpr int kColsPerBlock = 256;   // 32 lanes x 8 columns (one 16-byte load per lane and row)
constexpr int kWarps = 8;

// v -> a v + c for output feature n, from the chain's (linear) op list
__device__ __forceinline__ void linear_coeffs(const DevOps& ops, long long n, float& a, float& c) {
    a = 1.0f;
    c = 0.0f;
    for (int i = 0; i < ops.n; ++i) {
        const DevOp& op = ops.op[i];
        if (op.kind == FC_OP_BIAS_N) {
            c += load_scalar(op.p0, op.dt0, n);
        } else if (op.kind == FC_OP_AFFINE_N) {
            const float g = load_scalar(op.p0, op.dt0, n);
            a *= g;
            c = fmaf(c, g, load_scalar(op.p1, op.dt1, n));
        } else if (op.kind == FC_OP_SCALE) {
            a *= op.f0;
            c *= op.f0;
        }
    }
}

__device__ __forceinline__ void widen8(const uint4 w, bool f16, float (&v)[8]) {
    const uint32_t x[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float2 t = unpack16x2(x[j], f16);
        v[2 * j] = t.x;
        v[2 * j + 1] = t.y;
    }
}

// The two kernels behind the weight pass are launched with programmatic stream serialization: their CTAs are
// scheduled while the kernel in front drains, and wait here until that kernel has completed and its writes are
// visible (a no-op under an ordinary launch).
__device__ __forceinline__ void wait_for_previous_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// (Releasing the next kernel early, griddepcontrol.launch_dependents at the top of each kernel, measured slightly
// slower than the implicit release at exit: 37.5 vs 37.3 us on 1024 x 8192 x 8192.)

__global__ void __launch_bounds__(kWarps * 32)
weight_colsum_kernel(const CollapseParams p, int rows_per_block) {
    __shared__ double part[kWarps][kColsPerBlock];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long k0 = (long long) blockIdx.x * kColsPerBlock + lane * 8;
    const long long n_begin = (long long) blockIdx.y * rows_per_block;
    const long long n_end = min(n_begin + rows_per_block, (long long) p.N);
    const bool f16 = p.in_dt == FC_F16;
    const bool in_range = k0 < p.K;   // K is a multiple of 8
    double acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.0;
    double csum = 0.0;
    const unsigned short* B = (const unsigned short*) p.B;
    // a warp takes 8 consecutive rows at a time: lanes 0..7 work out the rows' coefficients while all
    // lanes have the 8 row segments in flight
#pragma unroll 1
    for (long long n = n_begin + warp * 8; n < n_end; n += kWarps * 8) {
        uint4 w[8];
#pragma unroll
        for (int r = 0; r < 8; ++r)
            w[r] = (in_range && n + r < n_end) ? __ldg(reinterpret_cast<const uint4*>(B + (n + r) * p.K + k0)) : make_uint4(0u, 0u, 0u, 0u);
        float a = 0.0f, c = 0.0f;
        if (lane < 8 && n + lane < n_end) linear_coeffs(p.ops, n + lane, a, c);
        // the 8 rows are added up in fp32 (8 roundings of 2^-24 relative each), the long sum over all rows in fp64
        float g[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) g[j] = 0.0f;
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const float ar = __shfl_sync(0xffffffffu, a, r), cr = __shfl_sync(0xffffffffu, c, r);
            csum += (double) cr;
            float v[8];
            widen8(w[r], f16, v);
#pragma unroll
            for (int j = 0; j < 8; ++j) g[j] = fmaf(ar, v[j], g[j]);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] += (double) g[j];
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) part[warp][lane * 8 + j] = acc[j];
    __syncthreads();
    {
        const int col = threadIdx.x;   // 256 threads, 256 columns
        const long long k = (long long) blockIdx.x * kColsPerBlock + col;
        if (k < p.K) {
            double s = 0.0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) s += part[w][col];
            p.partial[(size_t) blockIdx.y * p.K + k] = s;
        }
    }
    if (blockIdx.x == 0) {
        __shared__ double cw[kWarps];
        if (lane == 0) cw[warp] = csum;   // every lane holds the same csum
        __syncthreads();
        if (threadIdx.x == 0) {
            double s = 0.0;
            for (int w = 0; w < kWarps; ++w) s += cw[w];
            p.cpart[blockIdx.y] = s;
        }
    }
}

template <class... Args>
cudaError_t launch_after(void (*kernel)(Args...), dim3 grid, dim3 block, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

__global__ void __launch_bounds__(256)
colsum_finish_kernel(const CollapseParams p, int splits) {
    wait_for_previous_kernel();
    const long long k = (long long) blockIdx.x * blockDim.x + threadIdx.x;
    if (k < p.K) {
        double s = 0.0;
        for (int i = 0; i < splits; ++i) s += p.partial[(size_t) i * p.K + k];
        p.u[k] = (float) s;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        double s = 0.0;
        for (int i = 0; i < splits; ++i) s += p.cpart[i];
        *p.cterm = s;
    }
}

constexpr int kDotWarps = 4;
constexpr int kDotThreads = kDotWarps * 32;

// A block of 128 threads takes kRows rows; thread t owns columns t*8 + 1024*j (j < kDotLoads) of each pass
// over K, keeps its slice of u in registers and reuses it for every row of the block.
template <int kRows, int kDotLoads>
__global__ void __launch_bounds__(kDotThreads)
row_dot_kernel(const CollapseParams p) {
    constexpr int kDotChunk = kDotThreads * 8 * kDotLoads;   // columns a block covers per pass
    __shared__ double red[kDotWarps][kRows];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long m0 = (long long) blockIdx.x * kRows;
    const bool f16 = p.in_dt == FC_F16;
    const unsigned short* A = (const unsigned short*) p.A;
    double acc[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) acc[r] = 0.0;
    wait_for_previous_kernel();   // u and the constant term come from the kernel in front
#pragma unroll 1
    for (long long kc = (long long) threadIdx.x * 8; kc < p.K; kc += kDotChunk) {
        float uu[kDotLoads][8];
#pragma unroll
        for (int j = 0; j < kDotLoads; ++j) {
            const long long i = kc + (long long) j * kDotThreads * 8;
            const bool in = i < p.K;   // K is a multiple of 8
            const float4 ua = in ? __ldg(reinterpret_cast<const float4*>(p.u + i)) : make_float4(0.f, 0.f, 0.f, 0.f);
            const float4 ub = in ? __ldg(reinterpret_cast<const float4*>(p.u + i + 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
            uu[j][0] = ua.x; uu[j][1] = ua.y; uu[j][2] = ua.z; uu[j][3] = ua.w;
            uu[j][4] = ub.x; uu[j][5] = ub.y; uu[j][6] = ub.z; uu[j][7] = ub.w;
        }
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            const long long m = m0 + r;
            uint4 w[kDotLoads];
#pragma unroll
            for (int j = 0; j < kDotLoads; ++j) {
                const long long i = kc + (long long) j * kDotThreads * 8;
                w[j] = (m < p.M && i < p.K) ? __ldg(reinterpret_cast<const uint4*>(A + m * p.K + i)) : make_uint4(0u, 0u, 0u, 0u);
            }
            double s = 0.0;
#pragma unroll
            for (int j = 0; j < kDotLoads; ++j) {
                // 8 products added up in fp32, the long sum over the row in fp64
                float v[8];
                widen8(w[j], f16, v);
                float g = 0.0f;
#pragma unroll
                for (int q = 0; q < 8; ++q) g = fmaf(v[q], uu[j][q], g);
                s += (double) g;
            }
            acc[r] += s;
        }
    }
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        double s = acc[r];
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (lane == 0) red[warp][r] = s;
    }
    __syncthreads();
    if (threadIdx.x < kRows && m0 + threadIdx.x < p.M) {
        double s = *p.cterm;
#pragma unroll
        for (int w = 0; w < kDotWarps; ++w) s += red[w][threadIdx.x];
        p.out[m0 + threadIdx.x] = (float) (s * (double) p.post);
    }
}

// Slabs of rows for the weight pass.  The workspace is laid out for about kMaxBlocks blocks in all (at least 8 rows per
// warp); the launcher uses as many slabs as fill the resident slots once (three blocks of 256 threads and 75
// registers per SM): one full wave.  640 blocks on 148 SMs were 1.44 waves, and the short second one cost 6 - 9 %
// (1024 x 8192 x 8192 from a cold L2: 46.2 us with 640 blocks, 42.0 with 416; 222 blocks 52.3, 296 44 - 46, 864 44.1).
constexpr int kMaxBlocks = 640, kBlocksPerSm = 3;
int colsum_splits(long long N, long long K) {
    const long long col_blocks = (K + kColsPerBlock - 1) / kColsPerBlock;
    long long splits = (kMaxBlocks + col_blocks - 1) / col_blocks;
    const long long max_splits = (N + 8 * kWarps - 1) / (8 * kWarps);
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    if (splits > 65535) splits = 65535;
    return (int) splits;
}
int colsum_splits_launched(long long N, long long K, int num_sms) {
    const long long col_blocks = (K + kColsPerBlock - 1) / kColsPerBlock;
    long long splits = (long long) num_sms * kBlocksPerSm / col_blocks;   // rounded down: never a second, short wave
    const long long room = colsum_splits(N, K);
    if (splits > room) splits = room;
    if (splits < 1) splits = 1;
    return (int) splits;
}

}  // namespace

// workspace: [splits][K] fp64 partial column sums | [splits] fp64 partial constants | C | u[K] fp32
size_t collapse_workspace_bytes(long long N, long long K) {
    const size_t splits = (size_t) colsum_splits(N, K);
    const size_t doubles = splits * (size_t) K + splits + 1;
    return (doubles * sizeof(double) + 255) / 256 * 256 + ((size_t) K * sizeof(float) + 255) / 256 * 256;
}

cudaError_t launch_collapse(const CollapseParams& p_in, void* workspace, int num_sms, cudaStream_t stream, int* launches) {
    CollapseParams p = p_in;
    int splits = colsum_splits_launched(p.N, p.K, num_sms);
    const int rows_per_block = (int) ((p.N + splits - 1) / splits);
    splits = (int) ((p.N + rows_per_block - 1) / rows_per_block);
    const size_t full_splits = (size_t) colsum_splits(p.N, p.K);
    p.partial = (double*) workspace;
    p.cpart = p.partial + full_splits * (size_t) p.K;
    p.cterm = p.cpart + full_splits;
    p.u = (float*) ((char*) workspace + ((full_splits * (size_t) p.K + full_splits + 1) * sizeof(double) + 255) / 256 * 256);
    const int col_blocks = (int) ((p.K + kColsPerBlock - 1) / kColsPerBlock);
    note_kernel("weight_colsum colsum_finish row_dot");
    weight_colsum_kernel<<<dim3(col_blocks, splits), kWarps * 32, 0, stream>>>(p, rows_per_block);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    *launches += 1;
    if ((e = launch_after(colsum_finish_kernel, dim3(col_blocks), dim3(256), stream, p, splits)) != cudaSuccess) return e;
    *launches += 1;
    if (p.M <= 2048) e = launch_after(row_dot_kernel<1, 8>, dim3((unsigned) p.M), dim3(kDotThreads), stream, p);
    else if (p.K <= 4096) e = launch_after(row_dot_kernel<4, 4>, dim3((unsigned) ((p.M + 3) / 4)), dim3(kDotThreads), stream, p);
    else e = launch_after(row_dot_kernel<4, 8>, dim3((unsigned) ((p.M + 3) / 4)), dim3(kDotThreads), stream, p);
    *launches += 1;
    return e;
}

}  // namespace fc
