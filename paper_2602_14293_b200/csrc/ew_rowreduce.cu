// Kernel (a): memory-bound elementwise chain with an optional row reduction (logsumexp, softmax, sum, max, mean),
// one pass over the data.
//
// The row kernels give a warp a whole row (a lane per 16-byte chunk and several rows per warp for rows of at most 256
// columns; a CTA per row from 10240 columns on).  A lane owns 16-byte chunks (8 values of 16 bits) at a fixed column
// stride, issues the loads of four chunks of the input and of the residual tensor before any arithmetic, applies the
// op list in packed fp32x2 registers, stores the result once, and folds the fp32 values (before the output rounding)
// into a running (max, sum) pair that one shuffle merge per row finishes: no block barrier in the row loop.  The
// per-column vectors are converted to fp32 once per CTA and kept in shared memory, de-interleaved so that the lanes'
// float4 reads hit distinct banks.
//
// Instantiations: the row kernels for op lists of the shape [scale] [bias | affine] [relu | gelu] [scale] [clamp]
// [add tensor] on 16-bit rows with 16-byte aligned tensors, and a generic interpreter (any op list, any N, any
// alignment, fp32 storage) that also serves chains without a reduction whose rows are shorter than 256 columns.
#include <atomic>
#include "dev_common.cuh"

namespace fc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kInterpreterWarpRowChunks = 1024;   // interpreter: rows up to 8192 columns get a warp, longer ones a CTA

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
    asm volatile("griddepcontrol.wait;" ::: "memory");   // programmatic launch: see ew_rows_kernel
    const long long N = p.N;
    const int ebytes = p.x_dt == FC_F32 ? 4 : 2;
    const int ybytes = p.y_dt == FC_F32 ? 4 : 2;
    const bool x_f16 = p.x_dt == FC_F16, y_f16 = p.y_dt == FC_F16;
    constexpr int kV = 8;  // columns per chunk
    const bool x_vec = ((reinterpret_cast<uintptr_t>(p.x) | (uintptr_t)(N * ebytes)) & 15) == 0;
    const bool y_vec = p.y && ((reinterpret_cast<uintptr_t>(p.y) | (uintptr_t)(N * ybytes)) & 15) == 0;
    const long long chunks = (N + kV - 1) / kV;

    // one 8-column chunk of row m: load, ops, reduction partials, store
    // `phase`: 0 the whole chunk; row softmax takes two passes over a row: 1 accumulates (max, sum) without
    // storing, 2 computes the values again (the row's inputs are still in L2), turns them into
    // exp(v - row_max) * inv_sum and stores
    auto chunk = [&](long long m, long long c, MaxSum& acc, float& psum, float& pmax, int phase, float row_max, float inv_sum) {
            const long long n0 = c * kV;
            const bool full = n0 + kV <= N;
            float v[kV];
            if (p.x_dt != FC_F32) {
                if (full && x_vec) {
                    const uint4 q = __ldg(reinterpret_cast<const uint4*>((const unsigned short*) p.x + m * N + n0));
                    const float2 a = unpack16x2(q.x, x_f16), b = unpack16x2(q.y, x_f16), c2 = unpack16x2(q.z, x_f16), d = unpack16x2(q.w, x_f16);
                    v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y; v[4] = c2.x; v[5] = c2.y; v[6] = d.x; v[7] = d.y;
                } else {
#pragma unroll
                    for (int j = 0; j < kV; ++j) v[j] = n0 + j < N ? load_scalar(p.x, p.x_dt, m * N + n0 + j) : 0.0f;
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
            if (phase == 2) {
#pragma unroll
                for (int j = 0; j < kV; ++j) v[j] = exp2_fast((v[j] - row_max) * kLog2e) * inv_sum;
            } else if (p.reduce == FC_RED_ROW_LOGSUMEXP || p.reduce == FC_RED_ROW_SOFTMAX) {
                float mx = -CUDART_INF_F;
#pragma unroll
                for (int j = 0; j < kV; ++j) mx = n0 + j < N ? fmaxf(mx, v[j]) : mx;
                if (mx != -CUDART_INF_F) {   // a chunk of -inf only (a masked stretch of the row) adds nothing
                    float s = 0.0f;
#pragma unroll
                    for (int j = 0; j < kV; ++j) s += n0 + j < N ? exp2_fast((v[j] - mx) * kLog2e) : 0.0f;
                    acc = ms_merge(acc, MaxSum{mx, s});
                }
            }
            if (p.reduce >= FC_RED_ROW_SUM) {
#pragma unroll
                for (int j = 0; j < kV; ++j)
                    if (n0 + j < N) {
                        psum += v[j];
                        pmax = fmaxf(pmax, v[j]);
                    }
            }
            if (p.y && phase != 1) {
                if (p.y_dt != FC_F32) {
                    unsigned short* yp = (unsigned short*) p.y + m * N + n0;
                    if (full && y_vec) {
                        uint4 q;
                        q.x = pack16x2(v[0], v[1], y_f16); q.y = pack16x2(v[2], v[3], y_f16);
                        q.z = pack16x2(v[4], v[5], y_f16); q.w = pack16x2(v[6], v[7], y_f16);
                        *reinterpret_cast<uint4*>(yp) = q;
                    } else {
#pragma unroll
                        for (int j = 0; j < kV; ++j)
                            if (n0 + j < N) yp[j] = (unsigned short) (pack16x2(v[j], 0.0f, y_f16) & 0xffffu);
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
    };

    if (p.reduce == FC_RED_NONE) {
        // No reduction: rows do not matter, so the threads of the whole grid walk the chunks of the whole
        // tensor in order (a row of 64 columns would otherwise keep 8 of a CTA's 256 threads busy).
        const long long stride = (long long) gridDim.x * kThreads;
        const long long dm = stride / chunks, dc = stride - dm * chunks;
        const long long g = (long long) blockIdx.x * kThreads + threadIdx.x;
        long long m = g / chunks, c = g - m * chunks;
        MaxSum acc = ms_identity();
        float psum = 0.0f, pmax = 0.0f;
        while (m < p.M) {
            chunk(m, c, acc, psum, pmax, 0, 0.0f, 0.0f);
            m += dm;
            c += dc;
            if (c >= chunks) { c -= chunks; ++m; }
        }
        return;
    }

    if (chunks <= kInterpreterWarpRowChunks) {
        // Rows of moderate length: a warp per row, the row's partial results merged by shuffles.  A CTA per row
        // would pay two block barriers and a memory round trip per row with nothing else in flight (16384 rows
        // of 4096 columns with an op list the row kernel does not take: 201 us against 182 us).
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        for (long long m = (long long) blockIdx.x * kWarps + warp; m < p.M; m += (long long) gridDim.x * kWarps) {
            MaxSum acc = ms_identity();
            float psum = 0.0f, pmax = -CUDART_INF_F;
            const int phase = p.reduce == FC_RED_ROW_SOFTMAX ? 1 : 0;
            for (long long c = lane; c < chunks; c += 32) chunk(m, c, acc, psum, pmax, phase, 0.0f, 0.0f);
            if (p.reduce == FC_RED_ROW_SOFTMAX) {
                const MaxSum t = ms_warp_reduce(acc);
                const float inv = 1.0f / t.s;
                for (long long c = lane; c < chunks; c += 32) chunk(m, c, acc, psum, pmax, 2, t.m, inv);
            } else if (p.reduce == FC_RED_ROW_LOGSUMEXP) {
                const MaxSum t = ms_warp_reduce(acc);
                if (lane == 0) p.red[m] = t.m + logf(t.s);
            } else {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    psum += __shfl_xor_sync(0xffffffffu, psum, o);
                    pmax = fmaxf(pmax, __shfl_xor_sync(0xffffffffu, pmax, o));
                }
                if (lane == 0) p.red[m] = p.reduce == FC_RED_ROW_MAX ? pmax : (p.reduce == FC_RED_ROW_MEAN ? psum / (float) N : psum);
            }
        }
        return;
    }

    for (long long m = blockIdx.x; m < p.M; m += gridDim.x) {
        MaxSum acc = ms_identity();
        float psum = 0.0f, pmax = -CUDART_INF_F;   // ROW_SUM / ROW_MEAN and ROW_MAX
        const int phase = p.reduce == FC_RED_ROW_SOFTMAX ? 1 : 0;
        for (long long c = threadIdx.x; c < chunks; c += kThreads) chunk(m, c, acc, psum, pmax, phase, 0.0f, 0.0f);
        if (p.reduce == FC_RED_ROW_SOFTMAX) {
            const MaxSum t = block_merge(acc, red);   // every thread gets the row's pair
            const float inv = 1.0f / t.s;
            for (long long c = threadIdx.x; c < chunks; c += kThreads) chunk(m, c, acc, psum, pmax, 2, t.m, inv);
        } else if (p.reduce == FC_RED_ROW_LOGSUMEXP) {
            const MaxSum t = block_merge(acc, red);
            if (threadIdx.x == 0) p.red[m] = t.m + logf(t.s);
        } else if (p.reduce >= FC_RED_ROW_SUM) {
            // the pair slots carry (max, plain sum) here
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                psum += __shfl_xor_sync(0xffffffffu, psum, o);
                pmax = fmaxf(pmax, __shfl_xor_sync(0xffffffffu, pmax, o));
            }
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
            __syncthreads();
            if (lane == 0) red[warp] = MaxSum{pmax, psum};
            __syncthreads();
            if (threadIdx.x == 0) {
                float ts = 0.0f, tm = -CUDART_INF_F;
                for (int w = 0; w < kWarps; ++w) {
                    ts += red[w].s;
                    tm = fmaxf(tm, red[w].m);
                }
                p.red[m] = p.reduce == FC_RED_ROW_MAX ? tm : (p.reduce == FC_RED_ROW_MEAN ? ts / (float) N : ts);
            }
        }
    }
}


// ------------------------------------------------------------------------------------ fast path
// bf16 rows, N a multiple of 8, 16-byte aligned: [bias | affine]? -> [relu | gelu]? -> [+ tensor]?
// -> [row logsumexp]?.  One WARP owns a whole row, so the row reduction is a per-lane online
// (max, sum) plus a single warp shuffle merge: no block-level synchronisation in the row loop.
// Lane l handles the 16-byte chunks l, l+32, ... (every warp-wide access covers 512 contiguous
// bytes).  The per-column
// vectors are converted to fp32 once per CTA and kept in shared memory.
struct EwFastParams {
    const uint4* x;         // [M][N/8]
    const uint4* res;       // [M][N/8] or null
    uint4* y;               // [M][N/8] or null
    float* lse;             // [M] or null
    const void* vec0; int vec0_dt;   // bias / gamma
    const void* vec1; int vec1_dt;   // beta
    long long M;
    int N;
    int red_kind;           // fc_reduce of the row reduction (when the kernel is built with one)
    int is_f16;             // x, residual and y are IEEE half instead of bf16
    float post_scale, post_lo, post_hi;   // ACT with kActPost: v = clamp(v * post_scale, lo, hi) after the activation
    int ragged;             // long rows whose length is no multiple of 8 (no per-column vectors): rows start anywhere, the
                            // aligned middle of each row goes in 16-byte chunks, up to 14 edge elements one by one
    int stash;              // row softmax: the row's exponentials wait in shared memory for the second pass
    int* status;            // device status word (debug build's address checks)
    long long dbg_trim;     // debug build: bytes by which the checks believe y to be shorter (testing)
    float pre_scale;        // a SCALE op in front of everything, folded into gamma (PRE is then always affine;
                            // vec0 == null means gamma = 1, vec1 == null means beta = 0)
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Debug build: the row kernels' streaming accesses, checked against the extents of x / the residual (M * N 16-bit
// elements) and of y (the same, less what a test trimmed off); see FC_DBG_IN.
#ifdef FC_DEBUG
#define LD_STREAM(ptr, base, prm) (FC_DBG_IN((ptr), 16, (base), (prm).M * (long long) (prm).N * 2, (prm).status, kSiteEwLoad) ? ld_stream(ptr) : make_uint4(0u, 0u, 0u, 0u))
#define ST_STREAM(ptr, v, prm) do { if (FC_DBG_IN((ptr), 16, (prm).y, (prm).M * (long long) (prm).N * 2 - (prm).dbg_trim, (prm).status, kSiteEwStore)) st_stream((ptr), (v)); } while (0)
#define ST_RESULT(prm, row, value) do { if (FC_DBG_IN(&(prm).lse[row], 4, (prm).lse, (prm).M * 4, (prm).status, kSiteEwResult)) (prm).lse[row] = (value); } while (0)
#else
#define LD_STREAM(ptr, base, prm) ld_stream(ptr)
#define ST_STREAM(ptr, v, prm) st_stream((ptr), (v))
#define ST_RESULT(prm, row, value) (prm).lse[row] = (value)
#endif

constexpr int kPreNone = 0, kPreBias = 1, kPreAffine = 2;
constexpr int kActNone = 0, kActRelu = 1, kActGeluFast = 3;
constexpr int kActPost = 4;   // flag on top of the activation: a scale and a clamp follow it (before the residual)
constexpr int kGroup = 4;   // chunks in flight per lane and tensor
constexpr int kMaxWarpRow = 24576;   // longest row of the warp-per-row kernel (its vectors' fp32 copies must fit shared memory)
constexpr int kNarrowRow = 256;      // up to here (with a row reduction) a lane per chunk, several rows per warp
constexpr int kLongRow = 10240;      // from here on a CTA per row (measured: the warp-per-row kernel wins at 8192, loses at 12280)

// One chunk (8 columns starting at column 8*c) of one row: ops in packed fp32x2, one 16-byte store,
// and the chunk's contribution to the running (max, sum) of the row (log2 domain).
// The values of one chunk (8 columns starting at column 8*c) after the ops, as four fp32 pairs.
// The per-column operands of chunk c (gamma or bias in a, beta in b) from the fp32 copies in shared memory ...
template <int PRE, bool MAY_BE_CONST>
__device__ __forceinline__ void vec_from_smem(const float* svec, int N, int c, float2 (&a)[4], float2 (&b)[4], float const_gamma) {
    if (MAY_BE_CONST && PRE == kPreAffine && svec == nullptr) {
        // a lone SCALE folded into the affine step: gamma is that factor, beta 0, nothing in shared memory
        a[0] = a[1] = a[2] = a[3] = make_float2(const_gamma, const_gamma);
        b[0] = b[1] = b[2] = b[3] = make_float2(0.0f, 0.0f);
    } else if (PRE != kPreNone) {
        // shared-memory layout: the first and the second four columns of every chunk in separate arrays, so
        // that consecutive lanes (consecutive chunks) read consecutive float4s: no bank conflicts
        const int chunks = N >> 3;
        const float4* sv = reinterpret_cast<const float4*>(svec);
        const float4 a0 = sv[c];
        const float4 a1 = sv[chunks + c];
        a[0] = make_float2(a0.x, a0.y); a[1] = make_float2(a0.z, a0.w); a[2] = make_float2(a1.x, a1.y); a[3] = make_float2(a1.z, a1.w);
        if (PRE == kPreAffine) {
            const float4 b0 = sv[2 * chunks + c];
            const float4 b1 = sv[3 * chunks + c];
            b[0] = make_float2(b0.x, b0.y); b[1] = make_float2(b0.z, b0.w); b[2] = make_float2(b1.x, b1.y); b[3] = make_float2(b1.z, b1.w);
        }
    }
}
// ... or straight from the 16-bit vectors in global memory (rows too long for copies in shared memory; the
// vectors are shared by all rows and stay in L1 / L2).  A folded SCALE multiplies gamma here.
template <int PRE>
__device__ __forceinline__ void vec_from_global(const EwFastParams& p, int c, float2 (&a)[4], float2 (&b)[4]) {
    if (PRE != kPreNone) {
        const float s = PRE == kPreAffine ? p.pre_scale : 1.0f;
        if (p.vec0) {
            const uint4 q = __ldg(reinterpret_cast<const uint4*>(p.vec0) + c);
            const bool h = p.vec0_dt == FC_F16;
            const float2 ss = make_float2(s, s);
            a[0] = __fmul2_rn(unpack16x2(q.x, h), ss); a[1] = __fmul2_rn(unpack16x2(q.y, h), ss);
            a[2] = __fmul2_rn(unpack16x2(q.z, h), ss); a[3] = __fmul2_rn(unpack16x2(q.w, h), ss);
        } else {
            a[0] = a[1] = a[2] = a[3] = make_float2(s, s);
        }
        if (PRE == kPreAffine) {
            if (p.vec1) {
                const uint4 q = __ldg(reinterpret_cast<const uint4*>(p.vec1) + c);
                const bool h = p.vec1_dt == FC_F16;
                b[0] = unpack16x2(q.x, h); b[1] = unpack16x2(q.y, h); b[2] = unpack16x2(q.z, h); b[3] = unpack16x2(q.w, h);
            } else {
                b[0] = b[1] = b[2] = b[3] = make_float2(0.0f, 0.0f);
            }
        }
    }
}

template <int PRE, int ACT_, bool RES_>
__device__ __forceinline__ void ew_values(const uint4 xq, const uint4 rq, const float2 (&a)[4], const float2 (&b)[4], bool f16,
                                          float2 (&v)[4], const EwFastParams& prm) {
    constexpr int ACT = ACT_ & 3;
    constexpr bool kPost = (ACT_ & kActPost) != 0;
    constexpr bool RES = RES_ && !kPost;   // with post ops the residual is added behind them, not inside the activation
    v[0] = unpack16x2(xq.x, f16);
    v[1] = unpack16x2(xq.y, f16);
    v[2] = unpack16x2(xq.z, f16);
    v[3] = unpack16x2(xq.w, f16);
    if (PRE == kPreAffine) {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = __ffma2_rn(v[j], a[j], b[j]);
    } else if (PRE == kPreBias) {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = __fadd2_rn(v[j], a[j]);
    }
    float2 r[4];
    if (RES_) {
        r[0] = unpack16x2(rq.x, f16);
        r[1] = unpack16x2(rq.y, f16);
        r[2] = unpack16x2(rq.z, f16);
        r[3] = unpack16x2(rq.w, f16);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float2 t = v[j];
        if (ACT == kActRelu) t = make_float2(t.x < 0.0f ? 0.0f : t.x, t.y < 0.0f ? 0.0f : t.y);
        if (ACT == kActGeluFast) {
            constexpr float k0 = 0.7978845608028654f, k1 = k0 * 0.044715f;
            const float2 t2 = __fmul2_rn(t, t);
            const float2 z = __fmul2_rn(t, __ffma2_rn(t2, make_float2(k1, k1), make_float2(k0, k0)));
            const float2 hv = __fmul2_rn(t, make_float2(0.5f, 0.5f));
            const float2 th = make_float2(tanh_fast(z.x), tanh_fast(z.y));
            t = __ffma2_rn(hv, th, RES ? __fadd2_rn(hv, r[j]) : hv);
        } else if (RES) {
            t = __fadd2_rn(t, r[j]);
        }
        if (kPost) {
            t = __fmul2_rn(t, make_float2(prm.post_scale, prm.post_scale));
            t = make_float2(fminf(fmaxf(t.x, prm.post_lo), prm.post_hi), fminf(fmaxf(t.y, prm.post_lo), prm.post_hi));
            if (RES_) t = __fadd2_rn(t, r[j]);
        }
        v[j] = t;
    }
}

// VEC: 0 vectors from shared memory, 1 from global memory, 2 from shared memory unless a lone SCALE made them
// constants (checked at run time; only the softmax instantiations pay for the check)
template <int PRE, int ACT, bool RES, bool LSE, bool STORE, int VEC = 0>
__device__ __forceinline__ void ew_chunk(const uint4 xq, const uint4 rq, const float* svec, int N, int c, uint4* yr,
                                         int red_kind, bool f16, float& run_m, float& run_s, uint4* stash_e, float* stash_m,
                                         const EwFastParams& prm) {
    float2 v[4], a[4], b[4];
    if (VEC == 1) vec_from_global<PRE>(prm, c, a, b); else vec_from_smem<PRE, VEC == 2>(svec, N, c, a, b, prm.pre_scale);
    ew_values<PRE, ACT, RES>(xq, rq, a, b, f16, v, prm);
    if (STORE) {
        uint4 q;
        q.x = pack16x2(v[0].x, v[0].y, f16); q.y = pack16x2(v[1].x, v[1].y, f16);
        q.z = pack16x2(v[2].x, v[2].y, f16); q.w = pack16x2(v[3].x, v[3].y, f16);
        ST_STREAM(yr + c, q, prm);
    }
    if (LSE && red_kind >= FC_RED_ROW_SUM) {
        // ROW_SUM / ROW_MEAN / ROW_MAX: plain running sum and maximum
        const float cm = fmaxf(fmaxf(fmaxf(v[0].x, v[0].y), fmaxf(v[1].x, v[1].y)),
                               fmaxf(fmaxf(v[2].x, v[2].y), fmaxf(v[3].x, v[3].y)));
        const float2 t = __fadd2_rn(__fadd2_rn(v[0], v[1]), __fadd2_rn(v[2], v[3]));
        run_m = fmaxf(run_m, cm);
        run_s += t.x + t.y;
    } else if (LSE) {
        const float cm = fmaxf(fmaxf(fmaxf(v[0].x, v[0].y), fmaxf(v[1].x, v[1].y)),
                               fmaxf(fmaxf(v[2].x, v[2].y), fmaxf(v[3].x, v[3].y)));
        const float nm = fmaxf(run_m, cm * kLog2e);
        // while everything seen so far is -inf (a masked stretch at the start of the lane's columns) the
        // exponents are taken against 0, so that -inf stays -inf instead of turning into -inf - -inf
        const float base = nm == -CUDART_INF_F ? 0.0f : nm;
        const float2 l2e = make_float2(kLog2e, kLog2e), mnm = make_float2(-base, -base);
        float2 cs = make_float2(0.0f, 0.0f);
        float2 ex[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 e = __ffma2_rn(v[j], l2e, mnm);
            ex[j] = make_float2(exp2_fast(e.x), exp2_fast(e.y));
            cs = __fadd2_rn(cs, ex[j]);
        }
        run_s = fmaf(run_s, exp2_fast(run_m - base), cs.x + cs.y);
        run_m = nm;
        if (stash_e) {
            // Row softmax: the exponentials (in (0, 1], taken against the running maximum at this chunk) wait in the
            // output's 16-bit type, the running maximum beside them; the second pass rescales by
            // 2^(this maximum - row maximum) / sum.  Two roundings of 2^-9 (bf16) relative at most.
            uint4 q;
            q.x = pack16x2(ex[0].x, ex[0].y, f16); q.y = pack16x2(ex[1].x, ex[1].y, f16);
            q.z = pack16x2(ex[2].x, ex[2].y, f16); q.w = pack16x2(ex[3].x, ex[3].y, f16);
            stash_e[c] = q;
            stash_m[c] = nm;
        }
    }
}

// SOFTMAX (with LSE and without STORE): the row's values are turned into probabilities in a second pass.  Its own
// instantiations, with twice the registers: the second pass does not fit the 64 of the others without spilling.
template <int PRE, int ACT, bool RES, bool LSE, bool STORE, bool SOFTMAX = false>
__global__ void __launch_bounds__(kThreads, SOFTMAX ? 2 : 4) ew_rows_kernel(const EwFastParams p) {
    extern __shared__ float svec[];   // PRE != none: vec0 as fp32 [N] (chunk halves de-interleaved), then vec1 [N]
    // Launched with programmatic stream serialization: the CTAs are scheduled while the kernel in front drains and
    // wait here, before their first access to global memory, until it has completed and its writes are visible.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int N = p.N;
    const bool const_vec = SOFTMAX && PRE == kPreAffine && !p.vec0 && !p.vec1;   // a lone SCALE: no vectors to copy
    const float* svec_or_null = const_vec ? nullptr : svec;
    if (PRE != kPreNone && !const_vec) {
        // Every CTA converts the vectors once.  This prologue is a fixed cost of the launch (it measured 8 us
        // with one scalar load per column and thread): 16-bit vectors that are 16-byte aligned are read
        // eight columns per load, all loads of a thread issued before the first conversion.
        const int nchunks = N >> 3;
        float4* sv = reinterpret_cast<float4*>(svec);
        const bool fast0 = p.vec0 && p.vec0_dt != FC_F32 && (reinterpret_cast<uintptr_t>(p.vec0) & 15) == 0;
        const bool fast1 = PRE != kPreAffine || (p.vec1 && p.vec1_dt != FC_F32 && (reinterpret_cast<uintptr_t>(p.vec1) & 15) == 0);
        const bool plain = PRE != kPreAffine || p.pre_scale == 1.0f;   // a folded SCALE takes the scalar loop
        if (fast0 && fast1 && plain && nchunks <= 4 * kThreads) {
            uint4 q0[4], q1[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int c = threadIdx.x + k * kThreads;
                if (c < nchunks) {
                    q0[k] = __ldg(reinterpret_cast<const uint4*>(p.vec0) + c);
                    if (PRE == kPreAffine) q1[k] = __ldg(reinterpret_cast<const uint4*>(p.vec1) + c);
                }
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int c = threadIdx.x + k * kThreads;
                if (c < nchunks) {
                    const bool h0 = p.vec0_dt == FC_F16;
                    const float2 a = unpack16x2(q0[k].x, h0), b = unpack16x2(q0[k].y, h0), cc = unpack16x2(q0[k].z, h0), d = unpack16x2(q0[k].w, h0);
                    sv[c] = make_float4(a.x, a.y, b.x, b.y);
                    sv[nchunks + c] = make_float4(cc.x, cc.y, d.x, d.y);
                    if (PRE == kPreAffine) {
                        const bool h1 = p.vec1_dt == FC_F16;
                        const float2 e = unpack16x2(q1[k].x, h1), f = unpack16x2(q1[k].y, h1), g = unpack16x2(q1[k].z, h1), h = unpack16x2(q1[k].w, h1);
                        sv[2 * nchunks + c] = make_float4(e.x, e.y, f.x, f.y);
                        sv[3 * nchunks + c] = make_float4(g.x, g.y, h.x, h.y);
                    }
                }
            }
        } else {
            for (int i = threadIdx.x; i < N; i += kThreads) {
                // column i = chunk i/8, half (i%8)/4, element i%4  ->  float4 number half * chunks + chunk
                const int pos = ((((i >> 2) & 1) * nchunks) + (i >> 3)) * 4 + (i & 3);
                svec[pos] = (p.vec0 ? load_scalar(p.vec0, p.vec0_dt, i) : 1.0f) * (PRE == kPreAffine ? p.pre_scale : 1.0f);
                if (PRE == kPreAffine) svec[N + pos] = p.vec1 ? load_scalar(p.vec1, p.vec1_dt, i) : 0.0f;
            }
        }
        __syncthreads();
    }
    // Each warp walks whole rows, rows interleaved over all resident warps (measured: handing rows
    // out through a global counter evens out the CTAs' finish times but not the kernel's duration,
    // which is set by aggregate throughput).  Per row, a lane issues the loads of kGroup chunks of
    // the input and of the residual tensor (8 x 16 bytes in flight), then does their arithmetic.
    const int lane = threadIdx.x & 31;
    const int chunks = N >> 3;
    const int warp = threadIdx.x >> 5;
    const long long row_step = (long long) gridDim.x * kWarps;
    // row softmax: per warp N/8 chunks of eight 16-bit exponentials (16 bytes each), then N/8 running maxima
    uint4* stash_e = nullptr;
    float* stash_m = nullptr;
    if (SOFTMAX && p.stash) {
        float* base = svec + ((PRE == kPreNone || const_vec) ? 0 : (PRE == kPreAffine ? 2 : 1) * N);
        stash_e = reinterpret_cast<uint4*>(base) + (size_t) warp * chunks;
        stash_m = base + (size_t) kWarps * chunks * 4 + (size_t) warp * chunks;
    }
    for (long long row = (long long) blockIdx.x * kWarps + warp; row < p.M; row += row_step) {
        const uint4* xr = p.x + row * chunks;
        const uint4* rr = RES ? p.res + row * chunks : nullptr;
        uint4* yr = STORE ? p.y + row * chunks : nullptr;
        float run_m = -CUDART_INF_F, run_s = 0.0f;   // log2 domain: sum of 2^(y*log2e - run_m)
        // (softmax at 4096 columns, its rows waiting in shared memory: twice the loads in flight per lane gained 6 % while
        // the kernel ran one CTA per SM and lost 7 % at 1024 columns.  With two CTAs per SM, 128 registers per thread at
        // most, the eight chunks spill: 80 -> 121 us, as a second loop for long rows only too.  Left alone.)
        constexpr int kInFlight = kGroup;
        for (int c0 = lane; c0 < chunks; c0 += 32 * kInFlight) {
            uint4 xv[kInFlight], rv[kInFlight];
#pragma unroll
            for (int g = 0; g < kInFlight; ++g) {
                const int c = c0 + 32 * g;
                if (c < chunks) {
                    xv[g] = LD_STREAM(xr + c, p.x, p);
                    if (RES) rv[g] = LD_STREAM(rr + c, p.res, p);
                }
            }
#pragma unroll
            for (int g = 0; g < kInFlight; ++g) {
                const int c = c0 + 32 * g;
                if (c < chunks)
                    ew_chunk<PRE, ACT, RES, LSE, STORE, SOFTMAX ? 2 : 0>(xv[g], rv[g], svec_or_null, N, c, yr, SOFTMAX ? FC_RED_ROW_LOGSUMEXP : p.red_kind, p.is_f16 != 0, run_m, run_s,
                                                        SOFTMAX ? stash_e : nullptr, stash_m, p);
            }
        }
        if (LSE && !SOFTMAX && p.red_kind >= FC_RED_ROW_SUM) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                run_s += __shfl_xor_sync(0xffffffffu, run_s, o);
                run_m = fmaxf(run_m, __shfl_xor_sync(0xffffffffu, run_m, o));
            }
            if (lane == 0)
                ST_RESULT(p, row, p.red_kind == FC_RED_ROW_MAX ? run_m : (p.red_kind == FC_RED_ROW_MEAN ? run_s / (float) N : run_s));
        } else if (LSE) {
            // merge the 32 per-lane pairs (log2 domain)
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float om = __shfl_xor_sync(0xffffffffu, run_m, o);
                const float os = __shfl_xor_sync(0xffffffffu, run_s, o);
                const float nm = fmaxf(run_m, om);
                const float sa = run_m == -CUDART_INF_F ? 0.0f : run_s * exp2_fast(run_m - nm);
                const float sb = om == -CUDART_INF_F ? 0.0f : os * exp2_fast(om - nm);
                run_s = sa + sb;
                run_m = nm;
            }
            if constexpr (SOFTMAX) {
                // Second pass over the row: the exponentials wait in shared memory (rows of up to some 8000 columns)
                // and are rescaled; else the inputs are read again, from L2 where they still are, the values
                // computed again and stored as 2^(v log2e - max) / sum.
                float inv;
                asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(run_s));
                const float2 l2e = make_float2(kLog2e, kLog2e), mnm = make_float2(-run_m, -run_m), inv2 = make_float2(inv, inv);
                uint4* pr = p.y + row * chunks;
                if (stash_e) {
                    for (int c = lane; c < chunks; c += 32) {
                        const uint4 q = stash_e[c];
                        const float cmx = stash_m[c];
                        // everything up to this chunk was -inf: its exponentials are zeros, any finite factor will do
                        const float f = cmx == -CUDART_INF_F ? 0.0f : exp2_fast(cmx - run_m) * inv;
                        const float2 f2 = make_float2(f, f);
                        const bool h = p.is_f16 != 0;
                        const float2 a = __fmul2_rn(unpack16x2(q.x, h), f2), b = __fmul2_rn(unpack16x2(q.y, h), f2);
                        const float2 cc = __fmul2_rn(unpack16x2(q.z, h), f2), d = __fmul2_rn(unpack16x2(q.w, h), f2);
                        uint4 o;
                        o.x = pack16x2(a.x, a.y, h); o.y = pack16x2(b.x, b.y, h);
                        o.z = pack16x2(cc.x, cc.y, h); o.w = pack16x2(d.x, d.y, h);
                        ST_STREAM(pr + c, o, p);
                    }
                } else {
                    for (int c0 = lane; c0 < chunks; c0 += 32 * kGroup) {
                        uint4 xv[kGroup], rv[kGroup];
#pragma unroll
                        for (int g = 0; g < kGroup; ++g) {
                            const int c = c0 + 32 * g;
                            if (c < chunks) {
                                xv[g] = __ldcg(xr + c);
                                if (RES) rv[g] = __ldcg(rr + c);
                            }
                        }
#pragma unroll
                        for (int g = 0; g < kGroup; ++g) {
                            const int c = c0 + 32 * g;
                            if (c < chunks) {
                                float2 v[4];
                                float2 va[4], vb[4];
                                vec_from_smem<PRE, true>(svec_or_null, N, c, va, vb, p.pre_scale);
                                ew_values<PRE, ACT, RES>(xv[g], rv[g], va, vb, p.is_f16 != 0, v, p);
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    const float2 e = __ffma2_rn(v[j], l2e, mnm);
                                    v[j] = __fmul2_rn(make_float2(exp2_fast(e.x), exp2_fast(e.y)), inv2);
                                }
                                uint4 q;
                                q.x = pack16x2(v[0].x, v[0].y, p.is_f16 != 0); q.y = pack16x2(v[1].x, v[1].y, p.is_f16 != 0);
                                q.z = pack16x2(v[2].x, v[2].y, p.is_f16 != 0); q.w = pack16x2(v[3].x, v[3].y, p.is_f16 != 0);
                                ST_STREAM(pr + c, q, p);
                            }
                        }
                    }
                }
            } else if (lane == 0) ST_RESULT(p, row, (run_m + log2f(run_s)) * kLn2);
        }
    }
}

// ------------------------------------------------------------------------------------ narrow rows
// Rows of at most 256 columns (at most 32 chunks) with a row reduction: a warp per row would leave most lanes
// idle (64 columns: 8 of 32).  Here a lane owns one chunk and a warp covers 32 / cpr rows at a time, cpr = chunks
// per row rounded up to a power of two; the row's (max, sum) pair is merged by xor shuffles inside its group of
// cpr lanes.  The whole row sits in registers across the warp, so row softmax needs no second pass.  kGroup row
// groups are in flight per warp.  Which reduction, and whether the main output is stored, is decided at run time:
// this kernel is instantiated per op pattern only.
template <int PRE, int ACT, bool RES>
__global__ void __launch_bounds__(kThreads, 4) ew_narrow_kernel(const EwFastParams p, int cpr_log2) {
    extern __shared__ float svec[];
    asm volatile("griddepcontrol.wait;" ::: "memory");   // programmatic launch: see ew_rows_kernel
    const int N = p.N, chunks = N >> 3;
    if (PRE != kPreNone) {
        for (int i = threadIdx.x; i < N; i += kThreads) {
            const int pos = ((((i >> 2) & 1) * chunks) + (i >> 3)) * 4 + (i & 3);   // de-interleaved, as in ew_rows_kernel
            svec[pos] = (p.vec0 ? load_scalar(p.vec0, p.vec0_dt, i) : 1.0f) * (PRE == kPreAffine ? p.pre_scale : 1.0f);
            if (PRE == kPreAffine) svec[N + pos] = p.vec1 ? load_scalar(p.vec1, p.vec1_dt, i) : 0.0f;
        }
        __syncthreads();
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cpr = 1 << cpr_log2, rows_per_warp = 32 >> cpr_log2;
    const int c = lane & (cpr - 1), sub = lane >> cpr_log2;
    const bool f16 = p.is_f16 != 0;
    const int kind = p.red_kind;
    const bool softmax = kind == FC_RED_ROW_SOFTMAX, plain = kind >= FC_RED_ROW_SUM;
    const bool store = p.y != nullptr && !softmax;
    const long long step = (long long) gridDim.x * kWarps * rows_per_warp * kGroup;
    for (long long base = ((long long) blockIdx.x * kWarps + warp) * rows_per_warp * kGroup; base < p.M; base += step) {
        uint4 xv[kGroup], rv[kGroup];
#pragma unroll
        for (int g = 0; g < kGroup; ++g) {
            const long long row = base + g * rows_per_warp + sub;
            if (row < p.M && c < chunks) {
                xv[g] = LD_STREAM(p.x + row * chunks + c, p.x, p);
                if (RES) rv[g] = LD_STREAM(p.res + row * chunks + c, p.res, p);
            }
        }
#pragma unroll
        for (int g = 0; g < kGroup; ++g) {
            const long long row = base + g * rows_per_warp + sub;
            const bool valid = row < p.M && c < chunks;
            float2 v[4], a[4], b[4];
            float m = -CUDART_INF_F, sum = 0.0f;
            if (valid) {
                vec_from_smem<PRE, false>(svec, N, c, a, b, 1.0f);
                ew_values<PRE, ACT, RES>(xv[g], rv[g], a, b, f16, v, p);
                if (store) {
                    uint4 q;
                    q.x = pack16x2(v[0].x, v[0].y, f16); q.y = pack16x2(v[1].x, v[1].y, f16);
                    q.z = pack16x2(v[2].x, v[2].y, f16); q.w = pack16x2(v[3].x, v[3].y, f16);
                    ST_STREAM(p.y + row * chunks + c, q, p);
                }
                const float cm = fmaxf(fmaxf(fmaxf(v[0].x, v[0].y), fmaxf(v[1].x, v[1].y)), fmaxf(fmaxf(v[2].x, v[2].y), fmaxf(v[3].x, v[3].y)));
                if (plain) {
                    const float2 t = __fadd2_rn(__fadd2_rn(v[0], v[1]), __fadd2_rn(v[2], v[3]));
                    m = cm;
                    sum = t.x + t.y;
                } else {
                    // log2 domain; a chunk of -inf only takes its exponents against 0
                    m = cm * kLog2e;
                    const float base2 = m == -CUDART_INF_F ? 0.0f : m;
                    const float2 l2e = make_float2(kLog2e, kLog2e), mb = make_float2(-base2, -base2);
                    float2 cs = make_float2(0.0f, 0.0f);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float2 e = __ffma2_rn(v[j], l2e, mb);
                        cs = __fadd2_rn(cs, make_float2(exp2_fast(e.x), exp2_fast(e.y)));
                    }
                    sum = cs.x + cs.y;
                }
            }
            // merge inside the row's group of cpr lanes (lanes without a chunk hold the neutral pair)
            for (int o = cpr >> 1; o > 0; o >>= 1) {
                const float om = __shfl_xor_sync(0xffffffffu, m, o), os = __shfl_xor_sync(0xffffffffu, sum, o);
                if (plain) {
                    sum += os;
                    m = fmaxf(m, om);
                } else {
                    const float nm = fmaxf(m, om);
                    const float sa = m == -CUDART_INF_F ? 0.0f : sum * exp2_fast(m - nm);
                    const float sb = om == -CUDART_INF_F ? 0.0f : os * exp2_fast(om - nm);
                    sum = sa + sb;
                    m = nm;
                }
            }
            if (softmax) {
                if (valid) {
                    float inv;
                    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(sum));
                    const float2 l2e = make_float2(kLog2e, kLog2e), mnm = make_float2(-m, -m), inv2 = make_float2(inv, inv);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float2 e = __ffma2_rn(v[j], l2e, mnm);
                        v[j] = __fmul2_rn(make_float2(exp2_fast(e.x), exp2_fast(e.y)), inv2);
                    }
                    uint4 q;
                    q.x = pack16x2(v[0].x, v[0].y, f16); q.y = pack16x2(v[1].x, v[1].y, f16);
                    q.z = pack16x2(v[2].x, v[2].y, f16); q.w = pack16x2(v[3].x, v[3].y, f16);
                    ST_STREAM(p.y + row * chunks + c, q, p);
                }
            } else if (c == 0 && row < p.M) {
                ST_RESULT(p, row, kind == FC_RED_ROW_LOGSUMEXP ? (m + log2f(sum)) * kLn2
                           : kind == FC_RED_ROW_MAX ? m : (kind == FC_RED_ROW_MEAN ? sum / (float) N : sum));
            }
        }
    }
}

// ------------------------------------------------------------------------------------ long rows
// Rows of many thousands of columns (a vocabulary): a warp per row would walk them 32 chunks at a time and the
// fp32 copies of the per-column vectors would not fit shared memory.  Here a whole CTA owns a row: thread t takes
// chunks t, t + 256, ...; the vectors are read from their 16-bit originals (L1 / L2 resident); the row's
// (max, sum) pairs are merged by warp shuffles and one shared-memory exchange.  Row softmax takes its second
// pass over the row's inputs from L2 and computes the values again.
template <int PRE, int ACT, bool RES, bool LSE, bool STORE, bool SOFTMAX>
__global__ void __launch_bounds__(kThreads, SOFTMAX ? 2 : 4) ew_longrow_kernel(const EwFastParams p) {
    __shared__ float2 red[kWarps];
    asm volatile("griddepcontrol.wait;" ::: "memory");   // programmatic launch: see ew_rows_kernel
    const int N = p.N;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool f16 = p.is_f16 != 0;
    const int kind = SOFTMAX ? FC_RED_ROW_LOGSUMEXP : p.red_kind;
    const bool plain_kind = kind >= FC_RED_ROW_SUM;
    // one element of the row (ragged rows only): value after the ops, from 2-byte loads
    auto edge_value = [&](long long e) -> float {
        uint4 xq = make_uint4((uint32_t) __ldg((const unsigned short*) p.x + e), 0u, 0u, 0u), rq = make_uint4(0u, 0u, 0u, 0u);
        if (RES) rq.x = (uint32_t) __ldg((const unsigned short*) p.res + e);
        float2 v[4], a[4], b[4];
        vec_from_global<PRE>(p, 0, a, b);   // no vectors on this path: constants
        ew_values<PRE, ACT, RES>(xq, rq, a, b, f16, v, p);
        return v[0].x;
    };
    for (long long row = blockIdx.x; row < p.M; row += gridDim.x) {
        // rows of a ragged tensor start anywhere: `head` elements up to the next 16-byte boundary, then whole chunks,
        // then `tail` elements (head = tail = 0 when N is a multiple of 8)
        const long long e0 = row * N;
        const int head = p.ragged ? (int) ((8 - (e0 & 7)) & 7) : 0;
        const int chunks = (N - head) >> 3, tail = N - head - 8 * chunks;
        const uint4* xr = reinterpret_cast<const uint4*>((const unsigned short*) p.x + e0 + head);
        const uint4* rr = RES ? reinterpret_cast<const uint4*>((const unsigned short*) p.res + e0 + head) : nullptr;
        uint4* yr = STORE ? reinterpret_cast<uint4*>((unsigned short*) p.y + e0 + head) : nullptr;
        float run_m = -CUDART_INF_F, run_s = 0.0f;
        const bool edge = (int) threadIdx.x < head + tail;
        const long long edge_e = e0 + ((int) threadIdx.x < head ? threadIdx.x : head + 8 * chunks + ((int) threadIdx.x - head));
        if (edge) {
            const float val = edge_value(edge_e);
            if (STORE) ((unsigned short*) p.y)[edge_e] = (unsigned short) (pack16x2(val, 0.0f, f16) & 0xffffu);
            if (LSE) {
                if (plain_kind) { run_m = val; run_s = val; }
                else if (val != -CUDART_INF_F) { run_m = val * kLog2e; run_s = 1.0f; }
            }
        }
        for (int c0 = threadIdx.x; c0 < chunks; c0 += kThreads * kGroup) {
            uint4 xv[kGroup], rv[kGroup];
#pragma unroll
            for (int g = 0; g < kGroup; ++g) {
                const int c = c0 + kThreads * g;
                if (c < chunks) {
                    xv[g] = LD_STREAM(xr + c, p.x, p);
                    if (RES) rv[g] = LD_STREAM(rr + c, p.res, p);
                }
            }
#pragma unroll
            for (int g = 0; g < kGroup; ++g) {
                const int c = c0 + kThreads * g;
                if (c < chunks) ew_chunk<PRE, ACT, RES, LSE, STORE, 1>(xv[g], rv[g], nullptr, N, c, yr, kind, f16, run_m, run_s, nullptr, nullptr, p);
            }
        }
        if (LSE) {
            const bool plain = plain_kind;   // running sum and maximum instead of a logsumexp pair
            auto merge = [plain](float& am, float& as, float bm, float bs) {
                if (plain) { as += bs; am = fmaxf(am, bm); return; }
                const float nm = fmaxf(am, bm);
                const float sa = am == -CUDART_INF_F ? 0.0f : as * exp2_fast(am - nm);
                const float sb = bm == -CUDART_INF_F ? 0.0f : bs * exp2_fast(bm - nm);
                as = sa + sb;
                am = nm;
            };
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) merge(run_m, run_s, __shfl_xor_sync(0xffffffffu, run_m, o), __shfl_xor_sync(0xffffffffu, run_s, o));
            __syncthreads();   // the previous row's readers are done with `red`
            if (lane == 0) red[warp] = make_float2(run_m, run_s);
            __syncthreads();
            run_m = red[0].x; run_s = red[0].y;
#pragma unroll
            for (int w = 1; w < kWarps; ++w) merge(run_m, run_s, red[w].x, red[w].y);
            if constexpr (SOFTMAX) {
                float inv;
                asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(run_s));
                const float2 l2e = make_float2(kLog2e, kLog2e), mnm = make_float2(-run_m, -run_m), inv2 = make_float2(inv, inv);
                uint4* pr = reinterpret_cast<uint4*>((unsigned short*) p.y + e0 + head);
                if (edge) {
                    const float val = edge_value(edge_e);
                    const float pe = exp2_fast(fmaf(val, kLog2e, -run_m)) * inv;
                    ((unsigned short*) p.y)[edge_e] = (unsigned short) (pack16x2(pe, 0.0f, f16) & 0xffffu);
                }
                for (int c0 = threadIdx.x; c0 < chunks; c0 += kThreads * kGroup) {
                    uint4 xv[kGroup], rv[kGroup];
#pragma unroll
                    for (int g = 0; g < kGroup; ++g) {
                        const int c = c0 + kThreads * g;
                        if (c < chunks) {
                            xv[g] = __ldcg(xr + c);
                            if (RES) rv[g] = __ldcg(rr + c);
                        }
                    }
#pragma unroll
                    for (int g = 0; g < kGroup; ++g) {
                        const int c = c0 + kThreads * g;
                        if (c < chunks) {
                            float2 v[4], va[4], vb[4];
                            vec_from_global<PRE>(p, c, va, vb);
                            ew_values<PRE, ACT, RES>(xv[g], rv[g], va, vb, f16, v, p);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const float2 e = __ffma2_rn(v[j], l2e, mnm);
                                v[j] = __fmul2_rn(make_float2(exp2_fast(e.x), exp2_fast(e.y)), inv2);
                            }
                            uint4 q;
                            q.x = pack16x2(v[0].x, v[0].y, f16); q.y = pack16x2(v[1].x, v[1].y, f16);
                            q.z = pack16x2(v[2].x, v[2].y, f16); q.w = pack16x2(v[3].x, v[3].y, f16);
                            ST_STREAM(pr + c, q, p);
                        }
                    }
                }
            } else if (threadIdx.x == 0) {
                ST_RESULT(p, row, kind == FC_RED_ROW_LOGSUMEXP ? (run_m + log2f(run_s)) * kLn2
                           : kind == FC_RED_ROW_MAX ? run_m : (kind == FC_RED_ROW_MEAN ? run_s / (float) N : run_s));
            }
        }
    }
}

}  // namespace

// Recognise [scale]? -> [bias | affine]? -> [relu | gelu]? -> [scale]? -> [clamp]? -> [add tensor]? and fill the
// fast-path parameters.
static bool match_fast(const EwParams& p, EwFastParams* f, int* pre, int* act, bool* res) {
    if (p.x_dt == FC_F32 || (p.y && p.y_dt != p.x_dt)) return false;
    if ((p.N % 8 != 0 && p.N < kLongRow) || p.N >= 0x40000000LL || p.M >= 0x7fffffffLL) return false;
    if ((reinterpret_cast<uintptr_t>(p.x) | reinterpret_cast<uintptr_t>(p.y)) & 15) return false;
    int i = 0;
    *pre = kPreNone; *act = kActNone; *res = false;
    f->vec0 = f->vec1 = nullptr; f->vec0_dt = f->vec1_dt = FC_F32; f->res = nullptr;
    f->pre_scale = 1.0f;
    const bool scaled = i < p.ops.n && p.ops.op[i].kind == FC_OP_SCALE;
    if (scaled) f->pre_scale = p.ops.op[i++].f0;
    if (i < p.ops.n && (p.ops.op[i].kind == FC_OP_BIAS_N || p.ops.op[i].kind == FC_OP_AFFINE_N)) {
        *pre = p.ops.op[i].kind == FC_OP_BIAS_N ? kPreBias : kPreAffine;
        f->vec0 = p.ops.op[i].p0; f->vec0_dt = p.ops.op[i].dt0;
        f->vec1 = p.ops.op[i].p1; f->vec1_dt = p.ops.op[i].dt1;
        ++i;
    }
    if (scaled) {
        // x * s (+ b)  or  (x * s) * g + b: an affine step whose gamma carries the factor
        if (*pre == kPreBias) { f->vec1 = f->vec0; f->vec1_dt = f->vec0_dt; f->vec0 = nullptr; f->vec0_dt = FC_F32; }
        *pre = kPreAffine;
    }
    if (i < p.ops.n && (p.ops.op[i].kind == FC_OP_RELU || p.ops.op[i].kind == FC_OP_GELU_TANH)) {
        // GELU in the one-MUFU form (tanh.approx: within 6e-6 of the exact value, see gelu_tanh).  The exp-based form
        // (ex2 + rcp) measured no slower while the SMs held their full clock, but with three MUFU operations per
        // element (73 % of that pipe's cycles) the chain followed the SM clock: under the power cap, 1.75 GHz, a
        // 16384 x 4096 step took 73.5 instead of 68.9 us.
        *act = p.ops.op[i].kind == FC_OP_RELU ? kActRelu : kActGeluFast;
        ++i;
    }
    // [scale]? [clamp]? behind the activation: one flag, with neutral values for the one that is absent.  Not
    // instantiated for the softmax and reduction-only kernels.
    f->post_scale = 1.0f; f->post_lo = -INFINITY; f->post_hi = INFINITY;
    if (i < p.ops.n && (p.ops.op[i].kind == FC_OP_SCALE || p.ops.op[i].kind == FC_OP_CLAMP)) {
        if (p.N > kNarrowRow && (p.reduce == FC_RED_ROW_SOFTMAX || (p.reduce != FC_RED_NONE && !p.y))) return false;
        if (p.ops.op[i].kind == FC_OP_SCALE) f->post_scale = p.ops.op[i++].f0;
        if (i < p.ops.n && p.ops.op[i].kind == FC_OP_CLAMP) { f->post_lo = p.ops.op[i].f0; f->post_hi = p.ops.op[i].f1; ++i; }
        *act |= kActPost;
    }
    if (i < p.ops.n && p.ops.op[i].kind == FC_OP_ADD_TENSOR) {
        if (p.ops.op[i].dt0 != p.x_dt || (reinterpret_cast<uintptr_t>(p.ops.op[i].p0) & 15)) return false;
        *res = true;
        f->res = (const uint4*) p.ops.op[i].p0;
        ++i;
    }
    if (i != p.ops.n) return false;
    f->ragged = p.N % 8 != 0;
    if (f->ragged && (f->vec0 || f->vec1 || p.reduce == FC_RED_NONE || (*act & kActPost))) return false;   // long-row kernel, no vectors
    if (p.N > kMaxWarpRow) {
        // only the CTA-per-row kernel takes rows this long: a row reduction, no post ops, 16-bit aligned vectors
        const bool vec_ok = (!f->vec0 || (f->vec0_dt != FC_F32 && (reinterpret_cast<uintptr_t>(f->vec0) & 15) == 0)) &&
                            (!f->vec1 || (f->vec1_dt != FC_F32 && (reinterpret_cast<uintptr_t>(f->vec1) & 15) == 0));
        if (p.reduce == FC_RED_NONE || (*act & kActPost) || !vec_ok) return false;
    }
    f->x = (const uint4*) p.x; f->y = (uint4*) p.y; f->lse = p.red; f->M = p.M; f->N = (int) p.N;
    f->status = p.status; f->dbg_trim = p.dbg_trim;
    f->red_kind = p.reduce;
    f->is_f16 = p.x_dt == FC_F16;
    return true;
}

template <int PRE, int ACT, bool RES>
static cudaError_t launch_fast(const EwFastParams& f_in, bool lse, bool store, int num_sms, cudaStream_t stream) {
    EwFastParams f = f_in;
    const bool const_vec = f.red_kind == FC_RED_ROW_SOFTMAX && PRE == kPreAffine && !f.vec0 && !f.vec1;
    size_t smem = (PRE == kPreNone || const_vec) ? 0 : (size_t) f.N * 4 * (PRE == kPreAffine ? 2 : 1);
    f.stash = 0;
    const size_t stash_bytes = (size_t) kWarps * (f.N / 8) * (16 + 4);   // per chunk: eight 16-bit values and a maximum
    if (f.red_kind == FC_RED_ROW_SOFTMAX && smem + stash_bytes <= 200 * 1024) {
        f.stash = 1;
        smem += stash_bytes;
    }
    // Rows of at most 256 columns with a row reduction: a lane per chunk, several rows per warp.
    if (lse && f.N <= kNarrowRow) {
        int cpr_log2 = 0;
        while ((1 << cpr_log2) < f.N / 8) ++cpr_log2;
        const int rows_per_cta = kWarps * (32 >> cpr_log2) * kGroup;
        long long want = (f.M + rows_per_cta - 1) / rows_per_cta;
        if (want > (long long) num_sms * 4) want = (long long) num_sms * 4;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned) want);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = PRE == kPreNone ? 0 : (size_t) f.N * 4 * (PRE == kPreAffine ? 2 : 1);
        cfg.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        note_kernel("ew_narrow");
        return cudaLaunchKernelEx(&cfg, ew_narrow_kernel<PRE, ACT, RES>, f, cpr_log2);
    }
    // Rows from kLongRow columns on (lists without the post ops, 16-bit vectors on 16-byte boundaries) go to the
    // kernel that gives a CTA to a row.
    if constexpr ((ACT & kActPost) == 0) {
        const bool vec_ok = (!f.vec0 || (f.vec0_dt != FC_F32 && (reinterpret_cast<uintptr_t>(f.vec0) & 15) == 0)) &&
                            (!f.vec1 || (f.vec1_dt != FC_F32 && (reinterpret_cast<uintptr_t>(f.vec1) & 15) == 0));
        if (lse && f.N >= kLongRow && vec_ok) {
            cudaLaunchConfig_t cfg = {};
            const bool sm = f.red_kind == FC_RED_ROW_SOFTMAX;
            const long long want = (long long) num_sms * (sm ? 2 : 4);
            cfg.gridDim = dim3((unsigned) (f.M < want ? f.M : want));
            cfg.blockDim = dim3(kThreads);
            cfg.stream = stream;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr.val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            note_kernel(f.ragged ? "ew_longrow_ragged" : "ew_longrow");
            if (sm) return cudaLaunchKernelEx(&cfg, ew_longrow_kernel<PRE, ACT, RES, true, false, true>, f);
            if (store) return cudaLaunchKernelEx(&cfg, ew_longrow_kernel<PRE, ACT, RES, true, true, false>, f);
            return cudaLaunchKernelEx(&cfg, ew_longrow_kernel<PRE, ACT, RES, true, false, false>, f);
        }
    }
    if (f.N > kMaxWarpRow) return cudaErrorInvalidValue;   // not reached: match_fast sends such chains elsewhere
    long long ctas = (f.M + kWarps - 1) / kWarps;
    int per_sm = smem > 0 ? (int) ((227 * 1024) / (smem + 1024)) : 4;   // 228 KB per SM, 1 KB of it reserved per CTA
    per_sm = per_sm > 4 ? 4 : (per_sm < 1 ? 1 : per_sm);
    // Two CTAs per resident slot, except for the softmax form: the second half of the grid starts as the first
    // finishes, which evens out the tail.  Measured back to back in one process, 16384 x 4096: the logsumexp chain
    // 69.9 us with one CTA per slot, 67.95 with two, 69.3 with three (a stand-alone copy of the kernel: 592 CTAs 68.8,
    // 740 74.2, 888 76.1, 1184 67.1, 1776 67.8, a CTA per 8 rows 68.1); the softmax chain 74.2 / 75.0 / 76.0.
    const int per_slot = f.red_kind == FC_RED_ROW_SOFTMAX ? 1 : 2;
    if (ctas > (long long) num_sms * per_sm * per_slot) ctas = (long long) num_sms * per_sm * per_slot;
    // the dynamic shared-memory limit of each instantiation is raised once per device, to the maximum
    static std::atomic<bool> raised[4][64];   // zero-initialised; set idempotently from any thread
    int dev = 0;
    cudaGetDevice(&dev);
    auto go = [&](auto kernel, int variant) -> cudaError_t {
        if (smem > 48 * 1024 && (dev < 0 || dev >= 64 || !raised[variant][dev].load(std::memory_order_acquire))) {
            cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
            if (e != cudaSuccess) return e;
            if (dev >= 0 && dev < 64) raised[variant][dev].store(true, std::memory_order_release);
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned) ctas);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kernel, f);
    };
    note_kernel(f.red_kind == FC_RED_ROW_SOFTMAX ? (f.stash ? "ew_rows_softmax_stash" : "ew_rows_softmax") : "ew_rows");
    if constexpr ((ACT & kActPost) == 0) {
        if (f.red_kind == FC_RED_ROW_SOFTMAX) return go(ew_rows_kernel<PRE, ACT, RES, true, false, true>, 3);
        if (lse && !store) return go(ew_rows_kernel<PRE, ACT, RES, true, false>, 1);
    }
    if (lse && store) return go(ew_rows_kernel<PRE, ACT, RES, true, true>, 0);
    return go(ew_rows_kernel<PRE, ACT, RES, false, true>, 2);
}

cudaError_t launch_ew_rowreduce(const EwParams& p, int num_sms, cudaStream_t stream, int* launches) {
    *launches += 1;
    EwFastParams f;
    int pre, act;
    bool res;
    const bool lse = p.reduce != FC_RED_NONE;   // any row reduction
    // the row kernels give a warp to a row: without a reduction, rows under 256 columns go to the flat walk instead
    const bool narrow = !lse && p.N < 256;
    if (!narrow && match_fast(p, &f, &pre, &act, &res) && (lse || p.y)) {
        const bool store = p.y != nullptr && p.reduce != FC_RED_ROW_SOFTMAX;   // softmax stores in its second pass
#define FC_EW_CASE(PRE_, ACT_)                                                                       \
    if (pre == (PRE_) && act == (ACT_))                                                              \
        return res ? launch_fast<(PRE_), (ACT_), true>(f, lse, store, num_sms, stream)              \
                   : launch_fast<(PRE_), (ACT_), false>(f, lse, store, num_sms, stream);
        FC_EW_CASE(kPreNone, kActNone) FC_EW_CASE(kPreNone, kActRelu)
        FC_EW_CASE(kPreBias, kActNone) FC_EW_CASE(kPreBias, kActRelu)
        FC_EW_CASE(kPreAffine, kActNone) FC_EW_CASE(kPreAffine, kActRelu)
        FC_EW_CASE(kPreNone, kActGeluFast) FC_EW_CASE(kPreBias, kActGeluFast) FC_EW_CASE(kPreAffine, kActGeluFast)
        FC_EW_CASE(kPreNone, kActNone | kActPost) FC_EW_CASE(kPreNone, kActRelu | kActPost)
        FC_EW_CASE(kPreBias, kActNone | kActPost) FC_EW_CASE(kPreBias, kActRelu | kActPost)
        FC_EW_CASE(kPreAffine, kActNone | kActPost) FC_EW_CASE(kPreAffine, kActRelu | kActPost)
        FC_EW_CASE(kPreNone, kActGeluFast | kActPost) FC_EW_CASE(kPreBias, kActGeluFast | kActPost) FC_EW_CASE(kPreAffine, kActGeluFast | kActPost)
#undef FC_EW_CASE
    }
    const bool precise = false;   // tanh.approx is accurate to 6e-6 here (see gelu_tanh)
    long long work = p.M;   // CTAs that can be kept busy: rows (a warp each up to 8192 columns), or 256-chunk slabs of the whole tensor
    if (lse && (p.N + 7) / 8 <= kInterpreterWarpRowChunks) work = (p.M + kWarps - 1) / kWarps;
    if (!lse) work = (p.M * ((p.N + 7) / 8) + kThreads - 1) / kThreads;
    long long grid = work < (long long) num_sms * 8 ? work : (long long) num_sms * 8;
    if (grid < 1) grid = 1;
    note_kernel(lse ? "ew_interpreter_rows" : "ew_interpreter_flat");
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned) grid);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return precise ? cudaLaunchKernelEx(&cfg, ew_generic_kernel<true>, p) : cudaLaunchKernelEx(&cfg, ew_generic_kernel<false>, p);
}

}  // namespace fc
