// Back-to-back linear layers with every hidden width <= 256, kept on chip from the first layer to the last:
//
//     h1 = ops1(x W1^T),  h2 = ops2(round16(h1) W2^T),  ...,  out = opsL(round16(h_{L-1}) WL^T)
//
// (the cross-layer fusion of the paper's Level-3 discussion: consecutive linear layers reuse the
// activations instead of writing and re-reading them).  CTA pairs (cluster of 2, tcgen05 cta_group::2) walk
// 256-row panels of x, 128 rows per CTA; each CTA loads its own rows and half of every weight tile, so a
// k-block costs an SM 16 KB + 16 KB of L2 traffic instead of 16 KB + 32 KB (the fill of shared memory,
// not the MMA, sets the pace of these kernels).  For a panel, layer 1 is an ordinary TMA-fed main loop over K; its epilogue applies the layer's ops to
// the fp32 accumulator rows in tensor memory, rounds to the 16-bit storage type and writes the rows into
// shared memory in exactly the layout the tensor core reads its A operand from (K-major, 128-byte rows,
// 128-byte swizzle, 64-column k-blocks).  Layer 2's MMAs then take A from there and only W2 through TMA,
// and so on; the last layer's epilogue stores to global memory.  Hidden activations never leave the SM.
//
// Per CTA, 576 threads: warp 0 = TMA producer (one lane), warp 1 = tensor-memory owner and MMA issuer
// (one lane, leader CTA only), warps 2..17 = epilogue, one accumulator row and a quarter of the layer's
// columns per thread (a panel's layers run one after the other, so what a panel waits for is the epilogue:
// sixteen warps hide its latencies better than eight did, 131 vs 146 us on a 131072-row case).  A panel is a sequence of units (layer, k-block); the producers and the MMA thread walk the
// same sequence through a ring of stages (A 16 KB + half a W tile of up to 16 KB each; layers after the
// first use only the W part).  Barriers that both CTAs feed (stage full, accumulator free, activations
// written) live in the leader; the leader's commits release stages and announce accumulators in both.
// Accumulators alternate between two 256-column buffers of tensor memory, so the last epilogue of one panel overlaps the first main loop of
// the next.  Every wait is bounded, as in the other tensor-core kernels.
#include <atomic>
#include "tc_common.cuh"

namespace fc {
namespace {

constexpr int kRows = 128;            // rows of x per CTA; the pair covers 2 * kRows
constexpr int kBK = 64;
constexpr int kMaxWidth = 256;
constexpr int kEpiWarps = 16;
constexpr int kMlpThreads = (2 + kEpiWarps) * 32;
constexpr int kEpi = kEpiWarps * 32;
constexpr int kStages = 4;
constexpr int kABytes = kRows * kBK * 2;                // 16 KB
constexpr int kBBytes = (kMaxWidth / 2) * kBK * 2;      // this CTA's half of a W tile: up to 16 KB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kActBytes = kRows * kMaxWidth * 2;        // 64 KB: 4 k-blocks of 128 rows x 128 bytes
constexpr int kVecFloats = 3 * kMaxWidth;
constexpr int kMlpSmem = kStages * kStageBytes + kActBytes + kVecFloats * 4 + 256 + 1024;

struct MlpCtrl {
    unsigned long long full[kStages];
    unsigned long long empty[kStages];
    unsigned long long tfull[2];
    unsigned long long tempty[2];
    unsigned long long act_ready;
    uint32_t tmem_base;
    int abort;
    int epi_ok;
};
static_assert(sizeof(MlpCtrl) <= 256, "control block");

__device__ __forceinline__ int round_up(int v, int m) { return (v + m - 1) / m * m; }

__global__ void __launch_bounds__(kMlpThreads, 1)
mlp_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW0,
              const __grid_constant__ CUtensorMap tmW1, const __grid_constant__ CUtensorMap tmW2,
              const __grid_constant__ CUtensorMap tmW3, const MlpParams p) {
    extern __shared__ uint8_t smem_raw[];
    // the same offsets in both CTAs of the pair: the MMA addresses the peer's tiles by this CTA's descriptors
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* act = smem + kStages * kStageBytes;
    float* svec = reinterpret_cast<float*>(act + kActBytes);
    MlpCtrl* ctrl = reinterpret_cast<MlpCtrl*>(act + kActBytes + kVecFloats * 4);
    volatile int* abort_flag = &ctrl->abort;
    const CUtensorMap* tmW[4] = {&tmW0, &tmW1, &tmW2, &tmW3};

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = ptx::cluster_ctarank();
    const bool leader = cta_rank == 0;
    const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int L = p.layers;
    const int panels = (p.M + 2 * kRows - 1) / (2 * kRows);   // pair-panels of 256 rows

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->full[s]), 1);    // the leader's arrive.expect_tx for both CTAs' bytes
            ptx::mbar_init(ptx::smem_u32(&ctrl->empty[s]), 1);   // the leader's commit
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->tfull[b]), 1);   // the leader's commit
            ptx::mbar_init(ptx::smem_u32(&ctrl->tempty[b]), 2 * kEpiWarps); // the epilogue warps of both CTAs
        }
        ptx::mbar_init(ptx::smem_u32(&ctrl->act_ready), 2 * kEpiWarps);     // the epilogue warps of both CTAs
        ctrl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmX);
        for (int l = 0; l < L; ++l) ptx::prefetch_tensormap(tmW[l]);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&ctrl->tmem_base), 2 * kMaxWidth);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync();   // the peer's barriers exist before anything is signalled on them
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    // launched with programmatic stream serialization: nothing below touches global memory before the kernel in
    // front has completed; everything above overlapped its tail
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // k-blocks of layer l: over K of x for the first layer, over the previous layer's width afterwards
    auto num_kb = [&](int l) { return l == 0 ? (p.K0 + kBK - 1) / kBK : (p.width[l - 1] + kBK - 1) / kBK; };
    // the MMA's N of layer l: the width padded to 16; each CTA brings in half of those rows of W_l per k-block
    auto n_pad = [&](int l) { return round_up(p.width[l], 16); };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int pn = pair_id; pn < panels && ok; pn += num_pairs) {
                const int row0 = (pn * 2 + (int) cta_rank) * kRows;
                for (int l = 0; l < L && ok; ++l) {
                    const int nkb = num_kb(l);
                    const int half_rows = n_pad(l) / 2;
                    const uint32_t my_bytes = (l == 0 ? kABytes : 0) + (uint32_t) half_rows * kBK * 2;
                    for (int kb = 0; kb < nkb; ++kb, ++it) {
                        const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
                        if (!(ok = wait_bar(ptx::smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, p.status))) break;
                        const uint32_t full = ptx::mapa(ptx::smem_u32(&ctrl->full[s]), 0);   // the leader's barrier
                        const uint32_t sa = ptx::smem_u32(smem + s * kStageBytes);
                        // the leader expects the bytes of both CTAs (equal amounts); the peer's copies signal the
                        // same barrier
                        if (leader) ptx::mbar_arrive_expect_tx(ptx::smem_u32(&ctrl->full[s]), 2 * my_bytes);
                        if (l == 0) ptx::tma_load_2d_pair(sa, &tmX, kb * kBK, row0, full);
                        ptx::tma_load_2d_pair(sa + kABytes, tmW[l], kb * kBK, (int) cta_rank * half_rows, full);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (leader && lane == 0) {
            uint32_t it = 0, g = 0, acts = 0;
            bool ok = true;
            for (int pn = pair_id; pn < panels && ok; pn += num_pairs) {
                for (int l = 0; l < L && ok; ++l, ++g) {
                    const uint32_t buf = g & 1u, use = g >> 1;
                    if (!(ok = wait_bar(ptx::smem_u32(&ctrl->tempty[buf]), (use & 1u) ^ 1u, abort_flag, p.status))) break;
                    if (l > 0) {
                        // the previous layer's rows are in shared memory of both CTAs (written by their epilogue warps)
                        if (!(ok = wait_bar(ptx::smem_u32(&ctrl->act_ready), acts & 1u, abort_flag, p.status))) break;
                        ++acts;
                    }
                    ptx::tc_fence_after();
                    const uint32_t d_tmem = tmem_base + buf * kMaxWidth;
                    const uint32_t idesc = ptx::idesc_f16kind_f32(2 * kRows, n_pad(l), p.in_dt == FC_F16 ? 0u : 1u);
                    const int nkb = num_kb(l);
                    for (int kb = 0; kb < nkb; ++kb, ++it) {
                        const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
                        if (!(ok = wait_bar(ptx::smem_u32(&ctrl->full[s]), ph, abort_flag, p.status))) break;
                        ptx::tc_fence_after();
                        const uint32_t sa = ptx::smem_u32(smem + s * kStageBytes);
                        const uint32_t a_addr = l == 0 ? sa : ptx::smem_u32(act + kb * kABytes);
                        const uint64_t da = ptx::smem_desc_k128(a_addr), db = ptx::smem_desc_k128(sa + kABytes);
#pragma unroll
                        for (int k = 0; k < kBK / 16; ++k)
                            ptx::tc_mma_f16_pair(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                        ptx::tc_commit_pair(ptx::smem_u32(&ctrl->empty[s]), 3);      // frees the stage in both CTAs
                    }
                    if (ok) ptx::tc_commit_pair(ptx::smem_u32(&ctrl->tfull[buf]), 3);   // accumulators ready in both CTAs
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps (both CTAs): warp w reads
        // TMEM lanes 32*(w%4).. (one accumulator row per thread) and one of kParts ranges of the layer's columns
        const int et = threadIdx.x - 64;            // 0..kEpi-1
        const int part = (warp - 2) >> 2;           // which of the kEpiWarps / 4 column ranges this warp handles
        constexpr int kParts = kEpiWarps / 4;
        const int row = (warp & 3) * 32 + lane;     // TMEM lane quarter = warp % 4
        const uint32_t lane_addr = (uint32_t) ((warp & 3) * 32) << 16;
        const bool f16 = p.in_dt == FC_F16;
        const bool out_vec = (reinterpret_cast<uintptr_t>(p.out) & 15) == 0 && (p.width[L - 1] & 7) == 0;
        const uint32_t tempty_leader = ptx::mapa(ptx::smem_u32(&ctrl->tempty[0]), 0);
        const uint32_t act_ready_leader = ptx::mapa(ptx::smem_u32(&ctrl->act_ready), 0);
        uint32_t g = 0;
        bool alive = true;
        for (int pn = pair_id; pn < panels && alive; pn += num_pairs) {
            const long long m = (long long) (pn * 2 + (int) cta_rank) * kRows + row;
            for (int l = 0; l < L; ++l, ++g) {
                const uint32_t buf = g & 1u, use = g >> 1;
                const DevOps& ops = p.seg[l];
                const int width = p.width[l];
                // this layer's per-column vectors (fp32) into shared memory; the barrier also keeps the previous
                // layer's readers ahead of the overwrite
                ptx::bar_sync(1, kEpi);
                {
                    int slot = 0;
                    for (int i = 0; i < ops.n && slot < 3; ++i) {
                        const DevOp& op = ops.op[i];
                        const int nvec = op.kind == FC_OP_BIAS_N ? 1 : (op.kind == FC_OP_AFFINE_N ? 2 : 0);
                        for (int k = 0; k < nvec && slot < 3; ++k, ++slot)
                            for (int c = et; c < kMaxWidth; c += kEpi)
                                svec[slot * kMaxWidth + c] = c < width ? load_scalar(k ? op.p1 : op.p0, k ? op.dt1 : op.dt0, c) : 0.0f;
                    }
                }
                if (et == 0) ctrl->epi_ok = wait_bar(ptx::smem_u32(&ctrl->tfull[buf]), use & 1u, abort_flag, p.status);
                ptx::bar_sync(1, kEpi);
                if (!*(volatile int*) &ctrl->epi_ok) { alive = false; break; }
                ptx::tc_fence_after();
                const uint32_t tacc = tmem_base + buf * kMaxWidth + lane_addr;
                const bool last = l == L - 1;
                const int npad = n_pad(l);
                // intermediate layers fill whole k-blocks of the next A operand: columns past the width are zeros
                const int cols = last ? width : round_up(width, kBK);
                const int span = last ? round_up((width + kParts - 1) / kParts, 16) : cols / kParts;   // columns per warp group (cols is a multiple of 64)
                const int c_begin = min(part * span, cols), c_end = min(c_begin + span, cols);
                // one pass over this thread's columns; `apply` is the layer's op list on 16 columns of the row
                auto sweep = [&](auto&& apply) {
                    for (int c0 = c_begin; c0 < c_end; c0 += 16) {
                        float v[16];
                        if (c0 < npad) {
                            uint32_t r[16];
                            ptx::tmem_ld_32x16_async(tacc + c0, r);
                            ptx::tmem_wait_ld(r);
#pragma unroll
                            for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
                            apply(v, c0);
#pragma unroll
                            for (int j = 0; j < 16; ++j) v[j] = c0 + j < width ? v[j] : 0.0f;
                        } else {
#pragma unroll
                            for (int j = 0; j < 16; ++j) v[j] = 0.0f;
                        }
                        if (last) {
                            if (m < p.M) store16(p.out, p.out_dt, out_vec, v, m, c0, width, DbgOut{(long long) p.M * width * (p.out_dt == FC_F32 ? 4 : 2), p.status});
                        } else {
                            // A-operand layout: k-block c0/64, row `row` of 128 bytes, 16-byte chunk j stored at j ^ (row & 7)
                            uint8_t* kb_base = act + (c0 >> 6) * kABytes + row * 128;
                            const int j0 = (c0 & 63) >> 3;
#pragma unroll
                            for (int q = 0; q < 2; ++q) {
                                uint4 w;
                                w.x = pack16x2(v[8 * q + 0], v[8 * q + 1], f16);
                                w.y = pack16x2(v[8 * q + 2], v[8 * q + 3], f16);
                                w.z = pack16x2(v[8 * q + 4], v[8 * q + 5], f16);
                                w.w = pack16x2(v[8 * q + 6], v[8 * q + 7], f16);
                                *reinterpret_cast<uint4*>(kb_base + (((j0 + q) ^ (row & 7)) << 4)) = w;
                            }
                        }
                    }
                };
                // exp-based GELU (1e-6) rather than tanh.approx (6e-6): a hidden activation is rounded to 16 bits
                // next, and every bit of error moves more values across a rounding boundary
                if (ops.fused.valid) {
                    const FusedOps f = ops.fused;   // in registers for the whole pass
                    sweep([&](float (&v)[16], int c0) { fused_ops16<true>(v, f, svec, kMaxWidth, c0, m, c0, width, width); });
                } else {
                    sweep([&](float (&v)[16], int c0) { apply_ops16<true>(v, ops, svec, kMaxWidth, c0, m, c0, width, width); });
                }
                ptx::tc_fence_before();
                if (!last) ptx::fence_proxy_async_smem();   // the rows just written are read by the MMA (async proxy)
                __syncwarp();
                if (lane == 0) {
                    if (!last) ptx::mbar_arrive_cluster(act_ready_leader);
                    ptx::mbar_arrive_cluster(tempty_leader + buf * 8);
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    ptx::tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // a wait expired: give copies and MMAs still in flight time to land before releasing memory
        const unsigned long long t0 = ptx::globaltimer();
        while (ptx::globaltimer() - t0 < 2000000ull) __nanosleep(1000);
    }
    ptx::cluster_sync();   // neither CTA leaves while the other may still read its tiles or signal its barriers
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, 2 * kMaxWidth);
    }
}

}  // namespace

cudaError_t launch_mlp_tc(const MlpParams& p, const CUtensorMap& tmX, const CUtensorMap* tmW, int num_sms, cudaStream_t stream,
                          int* launches) {
    static std::atomic<bool> attr_set[64];     // zero-initialised; filled idempotently from any thread
    static std::atomic<int> max_clusters[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
        if ((e = cudaFuncSetAttribute(mlp_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMlpSmem)) != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev].store(true, std::memory_order_release);
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // added for the launch itself, not for the occupancy query
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(kMlpThreads);
    cfg.dynamicSmemBytes = kMlpSmem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (dev >= 0 && dev < 64 && max_clusters[dev].load(std::memory_order_acquire) == 0) {
        cfg.gridDim = dim3(num_sms & ~1);
        int n = 0;
        if ((e = cudaOccupancyMaxActiveClusters(&n, mlp_tc_kernel, &cfg)) != cudaSuccess) return e;
        max_clusters[dev].store(n > 0 ? n : 1, std::memory_order_release);
    }
    const int panels = (p.M + 2 * kRows - 1) / (2 * kRows);
    int pairs = dev >= 0 && dev < 64 ? max_clusters[dev].load(std::memory_order_acquire) : num_sms / 2;
    if (pairs > num_sms / 2) pairs = num_sms / 2;
    if (pairs > panels) pairs = panels;
    cfg.gridDim = dim3(2 * pairs);
    const CUtensorMap& w1 = tmW[p.layers > 1 ? 1 : 0];
    const CUtensorMap& w2 = tmW[p.layers > 2 ? 2 : 0];
    const CUtensorMap& w3 = tmW[p.layers > 3 ? 3 : 0];
    *launches += 1;
    cfg.numAttrs = 2;
    note_kernel("mlp_tc");
    return cudaLaunchKernelEx(&cfg, mlp_tc_kernel, tmX, tmW[0], w1, w2, w3, p);
}

}  // namespace fc
