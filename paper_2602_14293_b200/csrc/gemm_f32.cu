// Strict-fp32 GEMM NT (C = epilogue(A * B^T), A [M,K], B [N,K], all fp32) for small problems.
//
// fp32 FMA on the plain ALUs: a single-pass TF32 tensor-core product would miss the fp32 output
// tolerance, and at the sizes this path serves (hundreds per side) the run time is launch latency plus
// memory latency.  So the kernel is built to pay the memory latency once: a CTA owns a 16 x 32 output tile
// (256^3 gives 128 CTAs), and stages K through shared memory in slabs of 128 columns with cp.async, two
// slabs in flight from the first instruction on -- for K <= 256 every byte the CTA needs is requested
// before it computes anything.  128 threads x (2 x 2) outputs; a thread's rows are 8 apart and its columns
// 16 apart, so that its 16-byte shared-memory reads along K fall into distinct banks and its stores
// coalesce.  Rows are padded to 132 floats (33 x 16 bytes).
#include <atomic>
#include "dev_common.cuh"

namespace fc {
namespace {

constexpr int kTM = 16, kTN = 32;      // output tile
constexpr int kKS = 128;               // K columns per slab
constexpr int kPitch = kKS + 4;        // floats per shared-memory row
constexpr int kStages = 2;
constexpr int kGemmThreads = 128;
constexpr int kRows = kTM + kTN;       // rows of A and of B per slab
constexpr int kSmemBytes = kStages * kRows * kPitch * (int) sizeof(float);

__device__ __forceinline__ void cp_async16(float* dst, const float* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned) __cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory"); }

__global__ void __launch_bounds__(kGemmThreads) gemm_f32_kernel(const GemmF32Params p) {
    extern __shared__ __align__(16) float smem_f32[];
    // launched with programmatic stream serialization: scheduled while the kernel in front drains, and held here,
    // before the first access to global memory, until that kernel has completed
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;                   // columns tx, tx + 16; rows ty, ty + 8
    const int m0 = blockIdx.x * kTM, n0 = blockIdx.y * kTN;
    const bool vec = ((reinterpret_cast<uintptr_t>(p.A) | reinterpret_cast<uintptr_t>(p.B)) & 15) == 0 && (p.K & 3) == 0;
    const int slabs = (p.K + kKS - 1) / kKS;

    // rows 0..15 of a stage hold A's tile, rows 16..47 B's; 48 rows x 32 chunks of 4 floats = 12 per thread
    auto fill = [&](int slab) {
        float* stage = smem_f32 + (slab % kStages) * kRows * kPitch;
        const int k0 = slab * kKS;
#pragma unroll     // (not unrolled, the copies are issued more slowly: 256^3 12.5 instead of 11.1 us from a cold L2)
        for (int i = 0; i < kRows * (kKS / 4) / kGemmThreads; ++i) {
            const int c = tid + i * kGemmThreads;
            const int row = c >> 5, k = k0 + (c & 31) * 4;
            const bool is_a = row < kTM;
            const int grow = is_a ? m0 + row : n0 + row - kTM;
            const bool row_ok = grow < (is_a ? p.M : p.N);
            const float* src = (is_a ? p.A : p.B) + (long long) grow * p.K + k;
            float* dst = stage + row * kPitch + (c & 31) * 4;
            if (row_ok && vec && k + 3 < p.K) {
                cp_async16(dst, src);
            } else {
                float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
                if (row_ok) {
                    if (k + 0 < p.K) z.x = __ldg(src + 0);
                    if (k + 1 < p.K) z.y = __ldg(src + 1);
                    if (k + 2 < p.K) z.z = __ldg(src + 2);
                    if (k + 3 < p.K) z.w = __ldg(src + 3);
                }
                *reinterpret_cast<float4*>(dst) = z;
            }
        }
        cp_async_commit();
    };

    fill(0);
    if (slabs > 1) fill(1);
    float acc[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
    for (int s = 0; s < slabs; ++s) {
        if (s + 1 < slabs) cp_async_wait<1>(); else cp_async_wait<0>();
        __syncthreads();
        const float* stage = smem_f32 + (s % kStages) * kRows * kPitch;
        const float* a0p = stage + ty * kPitch;
        const float* a1p = stage + (ty + 8) * kPitch;
        const float* b0p = stage + (kTM + tx) * kPitch;
        const float* b1p = stage + (kTM + tx + 16) * kPitch;
#pragma unroll 8
        for (int k = 0; k < kKS; k += 4) {
            const float4 a0 = *reinterpret_cast<const float4*>(a0p + k), a1 = *reinterpret_cast<const float4*>(a1p + k);
            const float4 b0 = *reinterpret_cast<const float4*>(b0p + k), b1 = *reinterpret_cast<const float4*>(b1p + k);
            acc[0][0] = fmaf(a0.x, b0.x, acc[0][0]); acc[0][1] = fmaf(a0.x, b1.x, acc[0][1]);
            acc[1][0] = fmaf(a1.x, b0.x, acc[1][0]); acc[1][1] = fmaf(a1.x, b1.x, acc[1][1]);
            acc[0][0] = fmaf(a0.y, b0.y, acc[0][0]); acc[0][1] = fmaf(a0.y, b1.y, acc[0][1]);
            acc[1][0] = fmaf(a1.y, b0.y, acc[1][0]); acc[1][1] = fmaf(a1.y, b1.y, acc[1][1]);
            acc[0][0] = fmaf(a0.z, b0.z, acc[0][0]); acc[0][1] = fmaf(a0.z, b1.z, acc[0][1]);
            acc[1][0] = fmaf(a1.z, b0.z, acc[1][0]); acc[1][1] = fmaf(a1.z, b1.z, acc[1][1]);
            acc[0][0] = fmaf(a0.w, b0.w, acc[0][0]); acc[0][1] = fmaf(a0.w, b1.w, acc[0][1]);
            acc[1][0] = fmaf(a1.w, b0.w, acc[1][0]); acc[1][1] = fmaf(a1.w, b1.w, acc[1][1]);
        }
        __syncthreads();                       // everyone is done with this stage before it is refilled
        if (s + kStages < slabs) fill(s + kStages);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int m = m0 + ty + 8 * i;
        if (m >= p.M) continue;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int n = n0 + tx + 16 * j;
            if (n >= p.N) continue;
            float v[1] = {acc[i][j]};
            apply_ops<1, false>(v, p.ops, m, n, p.N, p.N);
            p.C[(long long) m * p.N + n] = v[0];
        }
    }
}

// Large problems (at least 96 tiles of 128 x 128): the classic register-tiled form.  256 threads x (8 x 8) outputs,
// as 2 x 2 blocks of 4 x 4 so that every shared-memory read is a 16-byte read without bank conflicts (64 FMAs per
// four reads); K in slabs of 16 through double-buffered shared memory, stored transposed ([k][row]) because both
// operands are K-major in global memory; the next slab is fetched into registers while this one is multiplied, one
// block barrier per slab.  Each output is still one fp32 FMA chain over ascending k.
constexpr int kBigTile = 128, kMidTile = 64, kBigSlab = 16;

// TILE = 128: as described; TILE = 64: one 4 x 4 block per thread (16 FMAs per two reads), for problems of fewer
// large tiles than keep the SMs busy.
template <int TILE>
__global__ void __launch_bounds__(256, TILE == 128 ? 2 : 4) gemm_f32_big_kernel(const GemmF32Params p) {
    constexpr int H = TILE / 64;            // 4 x 4 blocks per thread and dimension; rows lr + 64 h per loader thread
    constexpr int kPitch = TILE + 4;
    __shared__ __align__(16) float As[2][kBigSlab][kPitch];
    __shared__ __align__(16) float Bs[2][kBigSlab][kPitch];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * TILE, n0 = blockIdx.x * TILE;
    // loader mapping: 4 consecutive k of rows lr (and lr + 64), for A and for B
    const int lr = tid >> 2, lk = (tid & 3) * 4;
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
    auto park = [&](float (*dst)[kPitch], int row, const float4& r) {
        dst[lk + 0][row] = r.x; dst[lk + 1][row] = r.y; dst[lk + 2][row] = r.z; dst[lk + 3][row] = r.w;
    };

    float acc[4 * H][4 * H];
#pragma unroll
    for (int i = 0; i < 4 * H; ++i)
#pragma unroll
        for (int j = 0; j < 4 * H; ++j) acc[i][j] = 0.0f;

    float4 ra[H], rb[H];
#pragma unroll
    for (int h = 0; h < H; ++h) {
        ra[h] = load4(p.A, m0 + lr + 64 * h, p.M, lk);
        rb[h] = load4(p.B, n0 + lr + 64 * h, p.N, lk);
    }
#pragma unroll
    for (int h = 0; h < H; ++h) {
        park(As[0], lr + 64 * h, ra[h]);
        park(Bs[0], lr + 64 * h, rb[h]);
    }
    __syncthreads();
    int buf = 0;
    for (int k0 = 0; k0 < p.K; k0 += kBigSlab) {
        const bool more = k0 + kBigSlab < p.K;
        if (more) {
#pragma unroll
            for (int h = 0; h < H; ++h) {
                ra[h] = load4(p.A, m0 + lr + 64 * h, p.M, k0 + kBigSlab + lk);
                rb[h] = load4(p.B, n0 + lr + 64 * h, p.N, k0 + kBigSlab + lk);
            }
        }
#pragma unroll
        for (int k = 0; k < kBigSlab; ++k) {
            float a[4 * H], b[4 * H];
#pragma unroll
            for (int h = 0; h < H; ++h) {
                const float4 av = *reinterpret_cast<const float4*>(&As[buf][k][64 * h + ty * 4]);
                const float4 bv = *reinterpret_cast<const float4*>(&Bs[buf][k][64 * h + tx * 4]);
                a[4 * h] = av.x; a[4 * h + 1] = av.y; a[4 * h + 2] = av.z; a[4 * h + 3] = av.w;
                b[4 * h] = bv.x; b[4 * h + 1] = bv.y; b[4 * h + 2] = bv.z; b[4 * h + 3] = bv.w;
            }
#pragma unroll
            for (int i = 0; i < 4 * H; ++i)
#pragma unroll
                for (int j = 0; j < 4 * H; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (more) {
            // the other buffer was last read one slab ago, before the barrier that ended that slab
#pragma unroll
            for (int h = 0; h < H; ++h) {
                park(As[buf ^ 1], lr + 64 * h, ra[h]);
                park(Bs[buf ^ 1], lr + 64 * h, rb[h]);
            }
            __syncthreads();
            buf ^= 1;
        }
    }
    const bool c_vec = (reinterpret_cast<uintptr_t>(p.C) & 15) == 0 && (p.N & 3) == 0;
#pragma unroll
    for (int i = 0; i < 4 * H; ++i) {
        const int m = m0 + 64 * (i >> 2) + ty * 4 + (i & 3);
        if (m >= p.M) continue;
#pragma unroll
        for (int h = 0; h < H; ++h) {
            const int n = n0 + h * 64 + tx * 4;
            if (n >= p.N) continue;
            float v[4] = {acc[i][4 * h], acc[i][4 * h + 1], acc[i][4 * h + 2], acc[i][4 * h + 3]};
            apply_ops<4, false>(v, p.ops, m, n, p.N, p.N);
            float* c = p.C + (long long) m * p.N + n;
            if (c_vec && n + 3 < p.N) {
                *reinterpret_cast<float4*>(c) = make_float4(v[0], v[1], v[2], v[3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (n + j < p.N) c[j] = v[j];
            }
        }
    }
}

}  // namespace

cudaError_t launch_gemm_f32(const GemmF32Params& p, cudaStream_t stream, int* launches) {
    static std::atomic<bool> raised[64];   // zero-initialised; set idempotently from any thread
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !raised[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(gemm_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        raised[dev].store(true, std::memory_order_release);
    }
    const long long big_tiles = (long long) ((p.M + kBigTile - 1) / kBigTile) * ((p.N + kBigTile - 1) / kBigTile);
    // (1024^3 is 64 such tiles on 148 SMs: 137 us, against 77 us with 64 x 64 tiles)
    // (and not where an extent of at most 64 would leave half of every such tile empty)
    if (big_tiles >= 96 && p.M > kMidTile && p.N > kMidTile && (p.M + kBigTile - 1) / kBigTile <= 65535) {
        dim3 big((p.N + kBigTile - 1) / kBigTile, (p.M + kBigTile - 1) / kBigTile);
        note_kernel("gemm_f32_big");
        gemm_f32_big_kernel<kBigTile><<<big, 256, 0, stream>>>(p);
        *launches += 1;
        return cudaGetLastError();
    }
    // In between, from 512 tiles of 32 x 32 on, 64 x 64 tiles (768^3: 39 us, 1024^3: 77 us, 128 x 4096 x 4096: 191 us).
    // Below that the latency-oriented kernel wins (512^3: 20 against 27 us; 128 x 1024 x 1024: 21 against 50).
    const long long small_tiles = (long long) ((p.M + 31) / 32) * ((p.N + 31) / 32);
    if (small_tiles >= 512 && (p.M + kMidTile - 1) / kMidTile <= 65535) {
        dim3 mid((p.N + kMidTile - 1) / kMidTile, (p.M + kMidTile - 1) / kMidTile);
        note_kernel("gemm_f32_mid");
        gemm_f32_big_kernel<kMidTile><<<mid, 256, 0, stream>>>(p);
        *launches += 1;
        return cudaGetLastError();
    }
    dim3 grid((p.M + kTM - 1) / kTM, (p.N + kTN - 1) / kTN);   // M tiles in x (up to 2^31 - 1), N tiles in y (up to 65535)
    // a problem of one slab (K <= 128) asks for one stage only
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = p.K <= kKS ? kSmemBytes / kStages : kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    *launches += 1;
    note_kernel("gemm_f32");
    return cudaLaunchKernelEx(&cfg, gemm_f32_kernel, p);
}

}  // namespace fc
