// Device helpers shared by the kernels: bf16 packing, tanh-GELU, the epilogue op interpreter and
// (max, sum) pair algebra for online logsumexp / softmax.
#pragma once

#include <cuda_bf16.h>
#include <math_constants.h>

#include "fc_internal.h"

namespace fc {

// Debug build (-DFC_DEBUG): FC_DBG_IN(ptr, nbytes, base, bytes, status, site) is true when [ptr, ptr + nbytes) lies
// inside the tensor [base, base + bytes); otherwise it records FC_ERR_BOUNDS and the site in the status word and is
// false, and the caller skips the access.  In the ordinary build it is the constant true and costs nothing.
enum DbgSite { kSiteStore16 = 1, kSiteStoreRows = 2, kSiteSplitPark = 3, kSiteSplitMerge = 4, kSiteStats = 5, kSiteRowResult = 6,
               kSitePoolAvg = 7, kSitePoolMax = 8, kSitePoolStage = 9, kSiteEwLoad = 10, kSiteEwStore = 11, kSiteEwResult = 12 };
#ifdef FC_DEBUG
__device__ __forceinline__ bool dbg_in(const void* ptr, long long nbytes, const void* base, long long bytes, int* status, int site) {
    const long long off = (const char*) ptr - (const char*) base;
    const bool ok = base != nullptr && off >= 0 && off + nbytes <= bytes;
    if (!ok && status) atomicCAS(status, 0, FC_ERR_BOUNDS | (site << 8));
    return ok;
}
#define FC_DBG_IN(ptr, nbytes, base, bytes, status, site) ::fc::dbg_in((ptr), (nbytes), (base), (bytes), (status), (site))
#else
#define FC_DBG_IN(ptr, nbytes, base, bytes, status, site) true
#endif

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// two floats -> packed bf16x2 (lo in bits 0..15), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// 16-bit storage types: bf16 (FC_BF16) or IEEE half (FC_F16), two per 32-bit word
__device__ __forceinline__ float2 unpack16x2(uint32_t w, bool f16) {
    if (f16) {
        float2 r;
        asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tcvt.f32.f16 %0, lo;\n\tcvt.f32.f16 %1, hi;\n\t}" : "=f"(r.x), "=f"(r.y) : "r"(w));
        return r;
    }
    return make_float2(bf16_lo(w), bf16_hi(w));
}
__device__ __forceinline__ uint32_t pack16x2(float lo, float hi, bool f16) {
    uint32_t r;
    if (f16) asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    else asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ float tanh_fast(float x) {
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float exp2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// GELU, tanh form.  On sm_100a tanh.approx.f32 is far more accurate than its documented 2^-11 bound:
// measured over 4e8 points of [-12, 12] the result of this function differs from the fp64 value by at
// most 5.6e-6 (beyond that range tanh saturates to +-1 exactly), which is inside the fp32 output
// tolerance of 1e-4 (1 + |ref|) with a factor of 18 to spare, so every kernel uses the one-MUFU form.
// The exp-based form (ex2 + rcp, ~1e-6) stays available as kPrecise.
template <bool kPrecise>
__device__ __forceinline__ float gelu_tanh(float v) {
    const float z = 0.7978845608028654f * v * fmaf(0.044715f, v * v, 1.0f);
    if (kPrecise) {
        // 0.5 v (1 + tanh z) = v / (1 + exp(-2 z))
        const float e = exp2_fast(-2.0f * kLog2e * z);
        return __fdividef(v, 1.0f + e);
    } else {
        const float hv = 0.5f * v;
        return fmaf(hv, tanh_fast(z), hv);
    }
}


__device__ __forceinline__ float load_scalar(const void* p, int dt, long long i) {
    if (dt == FC_BF16) return __uint_as_float(((uint32_t) __ldg((const unsigned short*) p + i)) << 16);
    if (dt == FC_F16) return unpack16x2((uint32_t) __ldg((const unsigned short*) p + i), true).x;
    return __ldg((const float*) p + i);
}

// kN consecutive elements starting at element i of a tensor of type dt; elements from `valid` on are left at 0.
// Whole groups of eight elements on a 16-byte boundary are read with one (16-bit types) or two (fp32) vector
// loads per group (kN = 8 or 16).
template <int kN>
__device__ __forceinline__ void load_run(const void* p, int dt, long long i, long long valid, float (&out)[kN]) {
    if (kN % 8 == 0 && valid >= kN) {
        if (dt != FC_F32) {
            const unsigned short* q = (const unsigned short*) p + i;
            if ((reinterpret_cast<uintptr_t>(q) & 15) == 0) {
                const bool h = dt == FC_F16;
#pragma unroll
                for (int g = 0; g < kN / 8; ++g) {
                    const uint4 w = __ldg(reinterpret_cast<const uint4*>(q) + g);
                    const float2 a = unpack16x2(w.x, h), b = unpack16x2(w.y, h), c = unpack16x2(w.z, h), d = unpack16x2(w.w, h);
                    const int o = 8 * g;
                    out[(o + 0) % kN] = a.x; out[(o + 1) % kN] = a.y; out[(o + 2) % kN] = b.x; out[(o + 3) % kN] = b.y;
                    out[(o + 4) % kN] = c.x; out[(o + 5) % kN] = c.y; out[(o + 6) % kN] = d.x; out[(o + 7) % kN] = d.y;
                }
                return;
            }
        } else {
            const float* q = (const float*) p + i;
            if ((reinterpret_cast<uintptr_t>(q) & 15) == 0) {
#pragma unroll
                for (int g = 0; g < kN / 4; ++g) {
                    const float4 a = __ldg(reinterpret_cast<const float4*>(q) + g);
                    const int o = 4 * g;
                    out[(o + 0) % kN] = a.x; out[(o + 1) % kN] = a.y; out[(o + 2) % kN] = a.z; out[(o + 3) % kN] = a.w;
                }
                return;
            }
        }
    }
#pragma unroll
    for (int j = 0; j < kN; ++j) out[j] = j < valid ? load_scalar(p, dt, i + j) : 0.0f;
}

// Apply the op list to kN consecutive columns n0.. of row m (values in registers).
// `ld` is the row pitch (elements) of ADD_TENSOR operands; columns >= n_limit are not touched
// in memory (their register values are garbage-in, garbage-out and must not be stored).
template <int kN, bool kPreciseGelu>
__device__ __forceinline__ void apply_ops(float (&v)[kN], const DevOps& ops, long long m, long long n0,
                                          long long n_limit, long long ld) {
#pragma unroll 1
    for (int i = 0; i < ops.n; ++i) {
        const DevOp& op = ops.op[i];
        switch (op.kind) {
            case FC_OP_BIAS_N: {
                float b[kN];
                load_run<kN>(op.p0, op.dt0, n0, n_limit - n0, b);
#pragma unroll
                for (int j = 0; j < kN; ++j) v[j] += b[j];
                break;
            }
            case FC_OP_AFFINE_N: {
                float g[kN], b[kN];
                load_run<kN>(op.p0, op.dt0, n0, n_limit - n0, g);
                load_run<kN>(op.p1, op.dt1, n0, n_limit - n0, b);
#pragma unroll
                for (int j = 0; j < kN; ++j) v[j] = n0 + j < n_limit ? fmaf(v[j], g[j], b[j]) : v[j];
                break;
            }
            case FC_OP_RELU:
#pragma unroll
                for (int j = 0; j < kN; ++j) v[j] = v[j] < 0.0f ? 0.0f : v[j];
                break;
            case FC_OP_GELU_TANH:
#pragma unroll
                for (int j = 0; j < kN; ++j) v[j] = gelu_tanh<kPreciseGelu>(v[j]);
                break;
            case FC_OP_SCALE:
#pragma unroll
                for (int j = 0; j < kN; ++j) v[j] *= op.f0;
                break;
            case FC_OP_CLAMP:
#pragma unroll
                for (int j = 0; j < kN; ++j) v[j] = fminf(fmaxf(v[j], op.f0), op.f1);
                break;
            case FC_OP_ADD_TENSOR: {
                float t[kN];
                load_run<kN>(op.p0, op.dt0, m * ld + n0, n_limit - n0, t);
#pragma unroll
                for (int j = 0; j < kN; ++j) v[j] += t[j];
                break;
            }
            default:
                break;
        }
    }
}

// (max, sum of exp(v - max)) pairs.  Merge is associative and commutative.
struct MaxSum {
    float m, s;
};
__device__ __forceinline__ MaxSum ms_identity() { return MaxSum{-CUDART_INF_F, 0.0f}; }
__device__ __forceinline__ MaxSum ms_merge(MaxSum a, MaxSum b) {
    const float m = fmaxf(a.m, b.m);
    if (m == -CUDART_INF_F) return MaxSum{m, 0.0f};
    return MaxSum{m, a.s * exp2_fast((a.m - m) * kLog2e) + b.s * exp2_fast((b.m - m) * kLog2e)};
}
__device__ __forceinline__ MaxSum ms_warp_reduce(MaxSum a) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MaxSum b;
        b.m = __shfl_xor_sync(0xffffffffu, a.m, o);
        b.s = __shfl_xor_sync(0xffffffffu, a.s, o);
        a = ms_merge(a, b);
    }
    return a;
}

}  // namespace fc
