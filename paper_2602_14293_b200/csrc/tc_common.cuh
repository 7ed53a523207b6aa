// Device code shared by the tensor-core kernels: the bounded mbarrier wait and the epilogue's op list
// on 16 consecutive columns of one accumulator row.
#pragma once

#include "dev_common.cuh"
#include "ptx.cuh"

namespace fc {

// Bounded mbarrier wait.  Returns false if the CTA is aborting (this or another wait expired).
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = ptx::globaltimer();
    unsigned spins = 0;
    while (!ptx::mbar_try_wait(bar, parity)) {
        if ((++spins & 255u) == 0) {
            if (*abort_flag) return false;
            if (ptx::globaltimer() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                atomicExch(status, kStatusTimeout);
                return false;
            }
        }
    }
    return true;
}

// The op list applied to 16 consecutive columns (col0.. within the tile) of one row.  Per-column
// vectors come from the shared-memory slices staged for this tile (slot order = order of the
// vector operands in the op list); ADD_TENSOR reads global memory.
// The fused form of the op list on 16 consecutive columns, in packed fp32x2 arithmetic.
template <bool kPreciseGelu>
__device__ __forceinline__ void fused_ops16(float (&v)[16], const FusedOps& f, const float* svec, int bn, int col0,
                                            long long m, long long n0, long long n_limit, long long ld) {
    float2 w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) w[j] = make_float2(v[2 * j], v[2 * j + 1]);
    const float2 ps = make_float2(f.pre_scale, f.pre_scale);
    if (f.pre != 1 && f.pre_scale != 1.0f) {
#pragma unroll
        for (int j = 0; j < 8; ++j) w[j] = __fmul2_rn(w[j], ps);
    }
    if (f.pre != 0) {
        const float4* a = reinterpret_cast<const float4*>(svec + col0);
        if (f.pre == 1) {
            // (a SCALE in front of the bias rides in the same instruction: v * s + b)
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float4 t = a[q];
                w[2 * q] = __ffma2_rn(w[2 * q], ps, make_float2(t.x, t.y));
                w[2 * q + 1] = __ffma2_rn(w[2 * q + 1], ps, make_float2(t.z, t.w));
            }
        } else {
            const float4* b = reinterpret_cast<const float4*>(svec + bn + col0);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float4 g = a[q], t = b[q];
                w[2 * q] = __ffma2_rn(w[2 * q], make_float2(g.x, g.y), make_float2(t.x, t.y));
                w[2 * q + 1] = __ffma2_rn(w[2 * q + 1], make_float2(g.z, g.w), make_float2(t.z, t.w));
            }
        }
    }
    if (f.act == 2) {
        if (kPreciseGelu) {
            // gelu(t) * s = t * s / (1 + 2^(-2 z log2 e)),  z = sqrt(2/pi) (t + 0.044715 t^3)
            constexpr float k0 = -2.0f * kLog2e * 0.7978845608028654f, k1 = k0 * 0.044715f;
            const float2 sc = make_float2(f.scale, f.scale);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float2 t = w[j];
                const float2 e = __fmul2_rn(t, __ffma2_rn(__fmul2_rn(t, t), make_float2(k1, k1), make_float2(k0, k0)));
                const float2 d = __fadd2_rn(make_float2(exp2_fast(e.x), exp2_fast(e.y)), make_float2(1.0f, 1.0f));
                float2 inv;
                asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv.x) : "f"(d.x));
                asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv.y) : "f"(d.y));
                w[j] = __fmul2_rn(__fmul2_rn(t, sc), inv);
            }
        } else {
            // gelu(t) * s = h + h tanh(z) with h = (0.5 s) t
            constexpr float k0 = 0.7978845608028654f, k1 = k0 * 0.044715f;
            const float hs = 0.5f * f.scale;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float2 t = w[j];
                const float2 z = __fmul2_rn(t, __ffma2_rn(__fmul2_rn(t, t), make_float2(k1, k1), make_float2(k0, k0)));
                const float2 h = __fmul2_rn(t, make_float2(hs, hs));
                w[j] = __ffma2_rn(h, make_float2(tanh_fast(z.x), tanh_fast(z.y)), h);
            }
        }
    } else {
        if (f.act == 1) {
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = make_float2(w[j].x < 0.0f ? 0.0f : w[j].x, w[j].y < 0.0f ? 0.0f : w[j].y);
        }
        if (f.scale != 1.0f) {
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = __fmul2_rn(w[j], make_float2(f.scale, f.scale));
        }
    }
    if (f.clamp) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            w[j] = make_float2(fminf(fmaxf(w[j].x, f.lo), f.hi), fminf(fmaxf(w[j].y, f.lo), f.hi));
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) { v[2 * j] = w[j].x; v[2 * j + 1] = w[j].y; }
    if (f.res) {
        // this row's 16 columns of the residual: two 16-byte loads (16-bit storage) where the row allows it
        float t[16];
        load_run<16>(f.res_ptr, f.res_dt, m * ld + n0, n_limit - n0, t);
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] += t[j];
    }
}

template <bool kPreciseGelu>
__device__ __forceinline__ void apply_ops16(float (&v)[16], const DevOps& ops, const float* svec, int bn, int col0,
                                            long long m, long long n0, long long n_limit, long long ld) {
    if (ops.fused.valid) {
        fused_ops16<kPreciseGelu>(v, ops.fused, svec, bn, col0, m, n0, n_limit, ld);
        return;
    }
    int slot = 0;
#pragma unroll 1
    for (int i = 0; i < ops.n; ++i) {
        const DevOp& op = ops.op[i];
        switch (op.kind) {
            case FC_OP_BIAS_N: {
                const float4* b = reinterpret_cast<const float4*>(svec + slot * bn + col0);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float4 t = b[q];
                    v[4 * q] += t.x; v[4 * q + 1] += t.y; v[4 * q + 2] += t.z; v[4 * q + 3] += t.w;
                }
                ++slot;
                break;
            }
            case FC_OP_AFFINE_N: {
                const float4* g = reinterpret_cast<const float4*>(svec + slot * bn + col0);
                const float4* b = reinterpret_cast<const float4*>(svec + (slot + 1) * bn + col0);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float4 s = g[q], t = b[q];
                    v[4 * q] = fmaf(v[4 * q], s.x, t.x); v[4 * q + 1] = fmaf(v[4 * q + 1], s.y, t.y);
                    v[4 * q + 2] = fmaf(v[4 * q + 2], s.z, t.z); v[4 * q + 3] = fmaf(v[4 * q + 3], s.w, t.w);
                }
                slot += 2;
                break;
            }
            case FC_OP_RELU:
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = v[j] < 0.0f ? 0.0f : v[j];
                break;
            case FC_OP_GELU_TANH:
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = gelu_tanh<kPreciseGelu>(v[j]);
                break;
            case FC_OP_SCALE:
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] *= op.f0;
                break;
            case FC_OP_CLAMP:
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = fminf(fmaxf(v[j], op.f0), op.f1);
                break;
            case FC_OP_ADD_TENSOR: {
                float t[16];
                load_run<16>(op.p0, op.dt0, m * ld + n0, n_limit - n0, t);
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] += t[j];
                break;
            }
            default:
                break;
        }
    }
}

// 16 fp32 values of one row -> global memory as bf16 or fp32 (vector stores when aligned and in range)
// (debug build: `dbg` = the output's extent in bytes and the status word; a store that would leave it is skipped)
struct DbgOut {
    long long bytes;
    int* status;
};
__device__ __forceinline__ void store16(void* out, int out_dt, bool vec_ok, const float (&v)[16], long long m,
                                        long long n0, long long N, const DbgOut& dbg) {
#ifdef FC_DEBUG
    {
        const long long esz = out_dt != FC_F32 ? 2 : 4, cols = N - n0 < 16 ? N - n0 : 16;
        if (!FC_DBG_IN((const char*) out + (m * N + n0) * esz, cols * esz, out, dbg.bytes, dbg.status, kSiteStore16)) return;
    }
#endif
    if (out_dt != FC_F32) {
        const bool f16 = out_dt == FC_F16;
        unsigned short* o = (unsigned short*) out + m * N + n0;
        if (vec_ok && n0 + 16 <= N) {
            if ((reinterpret_cast<uintptr_t>(o) & 31) == 0) {
                // one 256-bit store: a whole 32-byte sector per thread and instruction
                asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(o), "r"(pack16x2(v[0], v[1], f16)),
                             "r"(pack16x2(v[2], v[3], f16)), "r"(pack16x2(v[4], v[5], f16)), "r"(pack16x2(v[6], v[7], f16)),
                             "r"(pack16x2(v[8], v[9], f16)), "r"(pack16x2(v[10], v[11], f16)), "r"(pack16x2(v[12], v[13], f16)),
                             "r"(pack16x2(v[14], v[15], f16))
                             : "memory");
                return;
            }
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                uint4 w;
                w.x = pack16x2(v[8 * q + 0], v[8 * q + 1], f16);
                w.y = pack16x2(v[8 * q + 2], v[8 * q + 3], f16);
                w.z = pack16x2(v[8 * q + 4], v[8 * q + 5], f16);
                w.w = pack16x2(v[8 * q + 6], v[8 * q + 7], f16);
                reinterpret_cast<uint4*>(o)[q] = w;
            }
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (n0 + j < N) o[j] = (unsigned short) (pack16x2(v[j], 0.0f, f16) & 0xffffu);
        }
    } else {
        float* o = (float*) out + m * N + n0;
        if (vec_ok && n0 + 16 <= N) {
            if ((reinterpret_cast<uintptr_t>(o) & 31) == 0) {
#pragma unroll
                for (int q = 0; q < 2; ++q)
                    asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(o + 8 * q), "f"(v[8 * q]), "f"(v[8 * q + 1]),
                                 "f"(v[8 * q + 2]), "f"(v[8 * q + 3]), "f"(v[8 * q + 4]), "f"(v[8 * q + 5]), "f"(v[8 * q + 6]), "f"(v[8 * q + 7])
                                 : "memory");
                return;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                reinterpret_cast<float4*>(o)[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (n0 + j < N) o[j] = v[j];
        }
    }
}

// Rows that do not start on 16-byte boundaries (N not a multiple of 8 for 16-bit outputs, of 4 for fp32): a thread
// storing its own row element by element makes every store instruction touch 32 sectors.  Here the warp's 32 x 16
// values go through shared memory (`stage`: 32 x 17 floats of this warp) and are written two rows per
// instruction, 16 consecutive elements each.  Every lane of the warp must call (`row_ok`: this lane's row exists).
__device__ __forceinline__ void store16_rows(void* out, int out_dt, float* stage, const float (&v)[16], long long m_lane0,
                                             long long M, long long n0, long long N, int lane, const DbgOut& dbg) {
#pragma unroll
    for (int j = 0; j < 16; ++j) stage[lane * 17 + j] = v[j];
    __syncwarp();
    const int c = lane & 15;
    if (n0 + c < N) {
#pragma unroll 4
        for (int it = 0; it < 16; ++it) {
            const int r = 2 * it + (lane >> 4);
            const long long row = m_lane0 + r;
            if (row < M && FC_DBG_IN((const char*) out + (row * N + n0 + c) * (out_dt == FC_F32 ? 4 : 2), out_dt == FC_F32 ? 4 : 2, out, dbg.bytes,
                                     dbg.status, kSiteStoreRows)) {
                const float x = stage[r * 17 + c];
                if (out_dt == FC_F32) ((float*) out)[row * N + n0 + c] = x;
                else ((unsigned short*) out)[row * N + n0 + c] = (unsigned short) (pack16x2(x, 0.0f, out_dt == FC_F16) & 0xffffu);
            }
        }
    }
    __syncwarp();
}

}  // namespace fc
