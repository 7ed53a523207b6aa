// Kernels (b), (c), (d): bf16 GEMM NT on the 5th-generation tensor cores (tcgen05.mma, fp32
// accumulators in tensor memory) fed by TMA, with the chain's epilogue applied in registers.
//
//   mode 0  out[m][n] = ops(acc)                               one bf16 / fp32 store per element
//   mode 1  row softmax over N fused across tiles: every tile publishes per-row (max, sum) of its
//           column slice, waits (bounded) until the row panel's tiles have all published, merges
//           the pairs and writes normalised probabilities straight from tensor memory
//   mode 2  implicit-GEMM convolution: the A operand is gathered by im2col-mode TMA from the NHWC
//           image (zero fill outside the image), B is the [Cout][R*S*Cin] weight matrix; the
//           epilogue applies ops (bias, ReLU) and sums each channel over the tile's pixels, adding
//           the scaled partial sums into out[image][channel]
//
// One persistent CTA per SM, 192 threads: warp 0 = TMA producer (one lane), warp 1 = MMA issuer
// (one lane) and owner of the tensor-memory allocation, warps 2..5 = epilogue (warp w reads TMEM
// lanes 32*(w%4)..).  A ring of kStages shared-memory stages (A 128x64, B BNx64, 128-byte swizzle)
// is handed over with full/empty mbarriers; two accumulator buffers in tensor memory let the
// epilogue of tile i overlap the main loop of tile i+1.  Every wait is bounded: on expiry the CTA
// records FC_ERR_TIMEOUT in the status word, stops storing and drains.
#include "dev_common.cuh"
#include "ptx.cuh"

namespace fc {
namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kThreads = 192;
constexpr int kEpiThreads = 128;
constexpr int kGroupM = 8;  // mode-0 raster: kGroupM row panels share each sweep over the columns

template <int BN>
struct Cfg {
    static constexpr int kABytes = BM * BK * 2;
    static constexpr int kBBytes = BN * BK * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStages = BN == 256 ? 4 : 6;
    static constexpr int kTmemCols = 2 * BN;
    static constexpr int kCtrlBytes = 256;
    static constexpr int kSmemBytes = kStages * kStageBytes + kCtrlBytes + 1024;  // 1024: alignment slack
};

struct Ctrl {
    unsigned long long full[8];
    unsigned long long empty[8];
    unsigned long long tfull[2];
    unsigned long long tempty[2];
    uint32_t tmem_base;
    int abort;
    int epi_ok[2];  // outcome of the epilogue's accumulator wait, one slot per accumulator buffer
};
static_assert(sizeof(Ctrl) <= 256, "control block");

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

__device__ __forceinline__ void tile_coords(int mode, int t, int tiles_m, int tiles_n, int& mb, int& nb) {
    if (mode == 0) {
        const int group = kGroupM * tiles_n;
        const int g = t / group, r = t - g * group;
        const int first = g * kGroupM;
        const int gm = min(kGroupM, tiles_m - first);
        mb = first + r % gm;
        nb = r / gm;
    } else {
        mb = t / tiles_n;  // panel-major: the tiles of one row panel are consecutive
        nb = t - mb * tiles_n;
    }
}

// Column sums over the 32 lanes of a warp for 32 columns held one per register: after the call
// lane j holds sum over lanes of v[j].  31 shuffles instead of 32 x 5.
__device__ __forceinline__ float warp_transpose_sum(float (&v)[32], int lane) {
#pragma unroll
    for (int half = 16; half >= 1; half >>= 1) {
        const bool upper = (lane & half) != 0;
#pragma unroll
        for (int i = 0; i < half; ++i) {
            const float send = upper ? v[i] : v[i + half];
            const float keep = upper ? v[i + half] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, half);
        }
    }
    return v[0];
}

template <int BN, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const TcParams p) {
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + C::kStages * C::kStageBytes);
    volatile int* abort_flag = &ctrl->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (p.M + BM - 1) / BM, tiles_n = (p.N + BN - 1) / BN;
    const int total_tiles = tiles_m * tiles_n;
    const int kb_per_tap = MODE == 2 ? (p.Cin + BK - 1) / BK : 0;
    const int num_kb = MODE == 2 ? p.R * p.S * kb_per_tap : (p.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->tfull[b]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->tempty[b]), 4);
        }
        ctrl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&ctrl->tmem_base), C::kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                int mb, nb;
                tile_coords(MODE == 0 ? 0 : 1, t, tiles_m, tiles_n, mb, nb);
                int img = 0, oh = 0, ow = 0;
                if constexpr (MODE == 2) {
                    const int pix = mb * BM, hw = p.OH * p.OW;
                    img = pix / hw;
                    const int rem = pix - img * hw;
                    oh = rem / p.OW;
                    ow = rem - oh * p.OW;
                }
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const uint32_t s = it % C::kStages, ph = (it / C::kStages) & 1u;
                    if (!(ok = wait_bar(ptx::smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, p.status))) break;
                    const uint32_t full = ptx::smem_u32(&ctrl->full[s]);
                    const uint32_t sa = ptx::smem_u32(smem + s * C::kStageBytes);
                    ptx::mbar_arrive_expect_tx(full, C::kStageBytes);
                    if constexpr (MODE == 2) {
                        const int tap = kb / kb_per_tap, c0 = (kb - tap * kb_per_tap) * BK;
                        const int r = tap / p.S, sx = tap - r * p.S;
                        ptx::tma_load_im2col_4d(sa, &tmA, c0, ow - p.pad, oh - p.pad, img, (uint16_t) sx, (uint16_t) r, full);
                        ptx::tma_load_2d(sa + C::kABytes, &tmB, tap * p.Cin + c0, nb * BN, full);
                    } else {
                        ptx::tma_load_2d(sa, &tmA, kb * BK, mb * BM, full);
                        ptx::tma_load_2d(sa + C::kABytes, &tmB, kb * BK, nb * BN, full);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_bf16_f32(BM, BN);
            uint32_t it = 0, tile_iter = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++tile_iter) {
                const uint32_t buf = tile_iter & 1u, aph = (tile_iter >> 1) & 1u;
                if (!(ok = wait_bar(ptx::smem_u32(&ctrl->tempty[buf]), aph ^ 1u, abort_flag, p.status))) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const uint32_t s = it % C::kStages, ph = (it / C::kStages) & 1u;
                    if (!(ok = wait_bar(ptx::smem_u32(&ctrl->full[s]), ph, abort_flag, p.status))) break;
                    ptx::tc_fence_after();
                    const uint32_t sa = ptx::smem_u32(smem + s * C::kStageBytes);
                    const uint64_t da = ptx::smem_desc_k128(sa), db = ptx::smem_desc_k128(sa + C::kABytes);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)  // 16 bf16 = 32 bytes per MMA along K -> +2 in 16-byte units
                        ptx::tc_mma_f16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                    ptx::tc_commit(ptx::smem_u32(&ctrl->empty[s]));
                }
                if (ok) ptx::tc_commit(ptx::smem_u32(&ctrl->tfull[buf]));
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int lane_grp = warp & 3;
        const int row = lane_grp * 32 + lane;
        const uint32_t lane_addr = (uint32_t) (lane_grp * 32) << 16;
        const bool precise = p.out_dt == FC_F32;
        const bool out_vec = (reinterpret_cast<uintptr_t>(p.out) & 15) == 0 && (p.N & 7) == 0;
        uint32_t tile_iter = 0;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, ++tile_iter) {
            int mb, nb;
            tile_coords(MODE == 0 ? 0 : 1, t, tiles_m, tiles_n, mb, nb);
            const uint32_t buf = tile_iter & 1u, aph = (tile_iter >> 1) & 1u;
            // one thread waits for the accumulator; its verdict reaches all four warps through shared
            // memory and a named barrier, so that they leave the loop together or not at all
            if (threadIdx.x == 64) ctrl->epi_ok[buf] = wait_bar(ptx::smem_u32(&ctrl->tfull[buf]), aph, abort_flag, p.status);
            ptx::bar_sync(2, kEpiThreads);
            if (!*(volatile int*) &ctrl->epi_ok[buf]) break;
            ptx::tc_fence_after();
            const uint32_t tacc = tmem_base + buf * BN + lane_addr;
            const long long m = (long long) mb * BM + row;
            const int n_tile = nb * BN;

            if constexpr (MODE == 0) {
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(tacc + c * 32, r);
                    const int n0 = n_tile + c * 32;
                    if (m < p.M && n0 < p.N) {
                        float v[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
                        if (precise) apply_ops<32, true>(v, p.ops, m, n0, p.N, p.N);
                        else apply_ops<32, false>(v, p.ops, m, n0, p.N, p.N);
                        if (p.out_dt == FC_BF16) {
                            unsigned short* o = (unsigned short*) p.out + m * p.N + n0;
                            if (out_vec && n0 + 32 <= p.N) {
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    uint4 w;
                                    w.x = pack_bf16x2(v[8 * q + 0], v[8 * q + 1]);
                                    w.y = pack_bf16x2(v[8 * q + 2], v[8 * q + 3]);
                                    w.z = pack_bf16x2(v[8 * q + 4], v[8 * q + 5]);
                                    w.w = pack_bf16x2(v[8 * q + 6], v[8 * q + 7]);
                                    reinterpret_cast<uint4*>(o)[q] = w;
                                }
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (n0 + j < p.N) o[j] = (unsigned short) (pack_bf16x2(v[j], 0.0f) & 0xffffu);
                            }
                        } else {
                            float* o = (float*) p.out + m * p.N + n0;
                            if (out_vec && n0 + 32 <= p.N) {
#pragma unroll
                                for (int q = 0; q < 8; ++q)
                                    reinterpret_cast<float4*>(o)[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (n0 + j < p.N) o[j] = v[j];
                            }
                        }
                    }
                }
            } else if constexpr (MODE == 1) {
                // pass 1: (max, sum) of this tile's slice of the row, online over 32-column chunks
                float mx = -CUDART_INF_F, sm = 0.0f;
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(tacc + c * 32, r);
                    const int n0 = n_tile + c * 32;
                    if (m < p.M && n0 < p.N) {
                        float v[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
                        apply_ops<32, false>(v, p.ops, m, n0, p.N, p.N);
                        float cm = -CUDART_INF_F;
#pragma unroll
                        for (int j = 0; j < 32; ++j) cm = n0 + j < p.N ? fmaxf(cm, v[j]) : cm;
                        const float nm = fmaxf(mx, cm);
                        float cs = 0.0f;
#pragma unroll
                        for (int j = 0; j < 32; ++j) cs += n0 + j < p.N ? exp2_fast((v[j] - nm) * kLog2e) : 0.0f;
                        sm = sm * exp2_fast((mx - nm) * kLog2e) + cs;
                        mx = nm;
                    }
                }
                if (m < p.M) __stcg(&p.stats[m * tiles_n + nb], make_float2(mx, sm));
                __threadfence();
                ptx::bar_sync(1, kEpiThreads);
                // one thread announces the tile and waits (bounded) for the panel's other tiles
                if (warp == 2 && lane == 0) {
                    ptx::red_release_gpu_add(&p.counters[mb], 1u);
                    const unsigned long long t0 = ptx::globaltimer();
                    unsigned spins = 0;
                    while (ptx::ld_acquire_gpu(&p.counters[mb]) < (unsigned) tiles_n) {
                        if ((++spins & 63u) == 0) {
                            if (*abort_flag) break;
                            if (ptx::globaltimer() - t0 > kWaitLimitNs) {
                                *abort_flag = 1;
                                atomicExch(p.status, kStatusTimeout);
                                break;
                            }
                        }
                    }
                    __threadfence();
                }
                ptx::bar_sync(1, kEpiThreads);
                const bool store = *abort_flag == 0;
                float row_m = -CUDART_INF_F, row_s = 0.0f;
                if (m < p.M && store) {
                    MaxSum a = ms_identity();
                    for (int j = 0; j < tiles_n; ++j) {
                        const float2 st = __ldcg(&p.stats[m * tiles_n + j]);
                        a = ms_merge(a, MaxSum{st.x, st.y});
                    }
                    row_m = a.m;
                    row_s = a.s;
                }
                const float inv = 1.0f / row_s, off = -row_m * kLog2e;
                // pass 2: normalise straight from tensor memory and store once
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(tacc + c * 32, r);
                    const int n0 = n_tile + c * 32;
                    if (m < p.M && n0 < p.N && store) {
                        float v[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
                        apply_ops<32, false>(v, p.ops, m, n0, p.N, p.N);
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = exp2_fast(fmaf(v[j], kLog2e, off)) * inv;
                        if (p.out_dt == FC_BF16) {
                            unsigned short* o = (unsigned short*) p.out + m * p.N + n0;
                            if (out_vec && n0 + 32 <= p.N) {
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    uint4 w;
                                    w.x = pack_bf16x2(v[8 * q + 0], v[8 * q + 1]);
                                    w.y = pack_bf16x2(v[8 * q + 2], v[8 * q + 3]);
                                    w.z = pack_bf16x2(v[8 * q + 4], v[8 * q + 5]);
                                    w.w = pack_bf16x2(v[8 * q + 6], v[8 * q + 7]);
                                    reinterpret_cast<uint4*>(o)[q] = w;
                                }
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (n0 + j < p.N) o[j] = (unsigned short) (pack_bf16x2(v[j], 0.0f) & 0xffffu);
                            }
                        } else {
                            float* o = (float*) p.out + m * p.N + n0;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (n0 + j < p.N) o[j] = v[j];
                        }
                    }
                }
            } else {
                // conv + global average pool: channel sums over this warp's 32 pixels
                const int hw = p.OH * p.OW;
                const long long pix_first = (long long) mb * BM + lane_grp * 32;
                const int img_first = (int) (pix_first / hw);
                const long long pix_last = min(pix_first + 31, (long long) p.M - 1);
                const int img_last = pix_last >= pix_first ? (int) (pix_last / hw) : img_first - 1;
                const int my_img = m < p.M ? (int) (m / hw) : -1;
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(tacc + c * 32, r);
                    const int n0 = n_tile + c * 32;
                    if (n0 >= p.N) continue;
                    float v[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
                    if (m < p.M) apply_ops<32, true>(v, p.ops, m, n0, p.N, p.N);
                    for (int img = img_first; img <= img_last; ++img) {
                        float w[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) w[j] = my_img == img ? v[j] : 0.0f;
                        const float s = warp_transpose_sum(w, lane);
                        if (n0 + lane < p.N) atomicAdd((float*) p.out + (long long) img * p.N + n0 + lane, s * p.inv_hw);
                    }
                }
            }
            // hand the accumulator buffer back to the MMA warp
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->tempty[buf]));
        }
    }

    // ---------------------------------------------------------------------- teardown
    ptx::tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // a wait expired: give copies and MMAs still in flight time to land before releasing memory
        const unsigned long long t0 = ptx::globaltimer();
        while (ptx::globaltimer() - t0 < 2000000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

template <int BN>
cudaError_t launch_bn(const TcParams& p, const CUtensorMap& tmA, const CUtensorMap& tmB, int grid, cudaStream_t stream) {
    const int smem = Cfg<BN>::kSmemBytes;
    cudaError_t e = cudaSuccess;
    switch (p.mode) {
        case 0:
            e = cudaFuncSetAttribute(gemm_tc_kernel<BN, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return e;
            gemm_tc_kernel<BN, 0><<<grid, kThreads, smem, stream>>>(tmA, tmB, p);
            break;
        case 1:
            e = cudaFuncSetAttribute(gemm_tc_kernel<BN, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return e;
            gemm_tc_kernel<BN, 1><<<grid, kThreads, smem, stream>>>(tmA, tmB, p);
            break;
        default:
            e = cudaFuncSetAttribute(gemm_tc_kernel<BN, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return e;
            gemm_tc_kernel<BN, 2><<<grid, kThreads, smem, stream>>>(tmA, tmB, p);
            break;
    }
    return cudaGetLastError();
}

}  // namespace

size_t gemm_tc_smem_bytes(int bn) { return bn == 256 ? Cfg<256>::kSmemBytes : Cfg<128>::kSmemBytes; }

cudaError_t launch_gemm_tc(const TcParams& p, const CUtensorMap& tmA, const CUtensorMap& tmB, int bn, int num_sms,
                           cudaStream_t stream, int* launches) {
    const int tiles = ((p.M + BM - 1) / BM) * ((p.N + bn - 1) / bn);
    const int grid = tiles < num_sms ? tiles : num_sms;
    *launches += 1;
    return bn == 256 ? launch_bn<256>(p, tmA, tmB, grid, stream) : launch_bn<128>(p, tmA, tmB, grid, stream);
}

}  // namespace fc
