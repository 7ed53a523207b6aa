// Kernels (b), (c), (d): bf16 GEMM NT on the 5th-generation tensor cores (tcgen05.mma, fp32
// accumulators in tensor memory) fed by TMA, with the chain's epilogue applied in registers.
//
//   mode 0  out[m][n] = ops(acc)                               one bf16 / fp32 store per element
//   mode 1  row softmax over N fused across tiles: every tile publishes per-row (max, sum) of its
//           column slice, waits (bounded) until the row panel's tiles have all published, merges
//           the pairs and writes normalised probabilities straight from tensor memory
//   mode 3  row logsumexp / sum / max / mean over N: as mode 0 (the main output is optional) plus per-tile
//           partial results; the tile that publishes last for a row panel merges them, so no tile waits
//   mode 2  implicit-GEMM convolution: the A operand is gathered by im2col-mode TMA from the NHWC
//           image (zero fill outside the image), B is the [Cout][R*S*Cin] weight matrix; the
//           epilogue applies ops (bias, ReLU) and sums each channel over the tile's pixels, adding
//           the scaled partial sums into out[image][channel]; or takes the maximum over 2x2 windows
//           into out[image][oh/2][ow/2][channel]
//   (template mode 4 is mode 2 for images of eight channels: a k-block then holds eight filter taps, gathered
//    as eight 8-channel copies into an unswizzled operand tile; a separate instantiation, so that the loops
//    of mode 2 stay as they are)
//   mode 6  mode 0 on block-scaled 8-bit operands (MXFP8: E4M3 elements, one E8M0 scale per row and 32 elements
//           along K).  tcgen05.mma.kind::mxf8f6f4.block_scale takes the scales from tensor memory: per k-block of
//           128 elements a 512-byte tile of A scales (this CTA's 128 rows x 4 blocks) and one of B scales (the
//           tile's 128 columns x 4 blocks) arrive with the operands (two more TMA loads from scale tiles that a
//           layout kernel has written, see launch_scale_tiles), tcgen05.cp moves them into four tensor-memory
//           columns each in front of the k-block's four MMAs, and MMA j names byte j of those columns.  Measured
//           layout: row r of the tile reads byte (r % 32) * 16 + (r / 32) * 4 + j of the 512; a B tile wider than 128
//           columns takes one such 512-byte tile (four more tensor-memory columns) per 128 columns.  Tiles are
//           256 x 240: two accumulator buffers of 240 columns and 12 scale columns share the 512 columns of tensor
//           memory (256 x 128 for N <= 128).  The epilogue's two warp groups take columns 0..127 and 128..239.
//
// Work unit: a 256 x BN output tile owned by a PAIR of CTAs on neighbouring SMs (cluster of 2,
// tcgen05 cta_group::2).  Each CTA loads its own 128 rows of A and HALF of the B tile, so a k-block
// costs each SM 16 KB + BN/2 * 128 B of L2 traffic instead of 16 KB + BN * 128 B; the leader CTA's
// MMA thread issues one 256 x BN x 16 MMA for both, and each CTA keeps the accumulator rows of its
// own 128 rows in its own tensor memory.  No TMA multicast is used anywhere.
//
// Per CTA, 320 threads: warp 0 = TMA producer (one lane), warp 1 = tensor-memory owner and, in the
// leader, MMA issuer (one lane), warps 2..9 = epilogue: warp w reads TMEM lanes 32*(w%4).. and the
// column half (w-2)/4 of the tile, so two warps per scheduler interleave their dependent chains.
// Shared-memory stages (A 128x64, B BN/2 x 64, 128-byte swizzle) are handed over with mbarriers:
// both producers signal the leader's "full" barrier, the leader's commit releases the stage in both
// CTAs.  Two accumulator buffers in tensor memory let the epilogue of tile i overlap the main loop
// of tile i+1.  Every wait is bounded: on expiry the CTA records FC_ERR_TIMEOUT in the status word,
// stops storing and drains.
//
// Split tiles.  When the tiles do not fill the last round of pairs (or there are fewer tiles than pairs
// at all: small-M GEMMs), the host cuts each tile of that round into `split` slices along K, one work
// unit each, all in that one round.  Every slice but the last parks its fp32 accumulator rows in scratch
// and bumps the tile's arrival counter; the last slice, which is given a few more k-blocks so that it
// finishes when the parked rows are there, waits (bounded) for the counter, adds the parked rows into
// its own accumulator in tensor memory and runs the epilogue as if it had done the whole tile.  The
// slices that park never wait, and every pair's split unit is its last one, so the wait cannot cycle.
//
// Arrival counters (split tiles, row panels) are handed back at zero: whoever observes the final count
// resets it, so a launch needs no memset as long as the previous one ran to completion.
#include "tc_common.cuh"

#include <atomic>
#include <cstdio>

namespace fc {
#ifdef FC_PROF
// Development aid, compiled out by default (build with -DFC_PROF=1 or 2): cycle accounting of the two single-thread
// roles of the leader CTA, per CTA pair.  Row = pair; columns: MMA thread total cycles, its waits for an accumulator
// buffer, unused, its waits for operand stages, k-blocks issued, cycles in MMA issue + commit, producer total cycles,
// producer waits for free stages, MMA thread total in nanoseconds (cycles / ns = the SM clock during the kernel).
__device__ long long g_prof[160][10];
__device__ long long g_prof_epi[160][8][8];   // per pair and tile: globaltimer at the epilogue's milestones (leader CTA, first thread)
__device__ long long g_prof_clk[160][8][8];   // the same milestones in SM cycles
#define EPI_MARK(i) do { if (et == 0 && leader && cluster_id < 160 && tile_iter < 8) { g_prof_epi[cluster_id][tile_iter][i] = (long long) ptx::globaltimer(); g_prof_clk[cluster_id][tile_iter][i] = clock64(); } } while (0)
#if FC_PROF >= 2   // per-wait accounting (itself costs about a hundred cycles per k-block)
#define PROF_T0(q) q = clock64()
#define PROF_ADD(acc, q) acc += clock64() - q
#else             // totals only
#define PROF_T0(q) (void) q
#define PROF_ADD(acc, q) (void) acc
#endif
#else
#define EPI_MARK(i) (void) 0
#define PROF_T0(q) (void) q
#define PROF_ADD(acc, q) (void) acc
#endif
namespace {

constexpr int BM = 128;          // rows per CTA; the pair covers 2 * BM
constexpr int BK = 64;
constexpr int kThreads = 320;
constexpr int kEpiThreads = 256;
constexpr int kMaxVecSlots = 3;  // per-column vectors staged in shared memory per tile

template <int BN>
struct Cfg {
    static constexpr int kABytes = BM * BK * 2;
    static constexpr int kBBytes = (BN / 2) * BK * 2;   // this CTA's half of the B tile
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStages = BN >= 240 ? 6 : 8;
    static constexpr int kTmemCols = 2 * BN;
    static constexpr int kVecBytes = 2 * kMaxVecSlots * BN * 4;   // double-buffered per-tile vector slices
    static constexpr int kCtrlBytes = 256;
    static constexpr int kPoolBytes = 8 * 32 * 17 * 4;   // max-pool: 32 pixels x 16 channels (+1 pad) per epilogue warp
    static constexpr int kXchgBytes = 2 * BM * 8;   // a (max, sum) pair per row and column half
    static constexpr int kSmemBytes = kStages * kStageBytes + kVecBytes + kCtrlBytes + kXchgBytes + kPoolBytes + 1024;  // + alignment slack
    // mode 6: per stage a 512-byte tile of A scales (this CTA's 128 rows) and one of B scales per 128 columns of the tile
    static constexpr int kScaleStage = 512 + 512 * ((BN + 127) / 128);
    static constexpr int kScaleBytes = kStages * kScaleStage;   // behind everything else
    static constexpr int kColHalf = BN == 240 ? 128 : BN / 2;   // columns of the first of the two epilogue warp groups
};

struct Ctrl {
    unsigned long long full[8];
    unsigned long long empty[8];
    unsigned long long tfull[2];
    unsigned long long tempty[2];
    uint32_t tmem_base;
    int abort;
    int epi_ok[2];  // outcome of the epilogue's accumulator wait, one slot per accumulator buffer
    int last;       // mode 3: this tile was the last of its row panel to publish
    int merge_ok;   // split tiles: the merging slice saw every other slice arrive
};
static_assert(sizeof(Ctrl) <= 256, "control block");

// pair-tile index -> (pair-panel index, column-tile index)
__device__ __forceinline__ void tile_coords(int mode, int group_m, int t, int tiles_m, int tiles_n, int& mb, int& nb) {
    if (mode == 0) {
        // raster: group_m pair-panels share each sweep over the column tiles, so that their rows of A
        // stay in L2 while B streams through once per group
        const int kGroupM = group_m;
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

// Work unit -> (tile, range of k-blocks).  Units below split_from are whole tiles; above it every tile is
// `split` consecutive units, one per slice of its k-blocks.
struct Unit {
    int tile, kb0, kb1, slice, nsl, v0;   // v0: index of the tile's first slice among the split units
};
__device__ __forceinline__ Unit unit_decode(int u, int split_from, int split, int split_kb, int num_kb) {
    Unit w;
    if (u < split_from || split <= 1) {
        w.tile = u; w.kb0 = 0; w.kb1 = num_kb; w.slice = 0; w.nsl = 1; w.v0 = 0;
    } else {
        const int v = u - split_from;
        const int ti = v / split;
        w.tile = split_from + ti;
        w.slice = v - ti * split;
        w.nsl = split;
        w.v0 = ti * split;
        w.kb0 = w.slice * split_kb;                                   // split_kb k-blocks per parking slice,
        w.kb1 = w.slice == split - 1 ? num_kb : w.kb0 + split_kb;     // the rest for the merging one
    }
    return w;
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

// One pass over this thread's half row of the accumulator in 16-column chunks: load, wait, f(c, r), which may change r
// and store it back; the first `live` chunks only (a 240-column tile's second half has seven: the eighth belongs to the
// other buffer).  A plain loop on purpose: a tcgen05.ld + wait takes 30 - 60 cycles, and neither keeping the next
// load in flight nor 32-column loads (two and four copies of f's code) measured faster than this single copy.
template <int kChunks, class F>
__device__ __forceinline__ void tmem_sweep(uint32_t tacc, int live, F&& f) {
#pragma unroll 1
    for (int c = 0; c < live; ++c) {
        uint32_t r[16];
        ptx::tmem_ld_32x16_async(tacc + c * 16, r);
        ptx::tmem_wait_ld(r);
        f(c, r);
    }
}

// Two chunks per iteration, the second load in flight while the first chunk is processed (the convolution's pooling sweeps).
template <int kChunks, class F>
__device__ __forceinline__ void tmem_sweep16(uint32_t tacc, F&& f) {
    uint32_t ra[16], rb[16];
    ptx::tmem_ld_32x16_async(tacc, ra);
#pragma unroll 1
    for (int c = 0; c < kChunks; c += 2) {
        ptx::tmem_wait_ld(ra);
        ptx::tmem_ld_32x16_async(tacc + (c + 1) * 16, rb);
        f(c, ra);
        ptx::tmem_wait_ld(rb);
        if (c + 2 < kChunks) ptx::tmem_ld_32x16_async(tacc + (c + 2) * 16, ra);
        f(c + 1, rb);
    }
}

// k-blocks of one tile.  Convolution: one block per (tap, 64-channel slice), or (a_packed, chosen by the caller for
// very few channels) blocks of eight 8-channel chunks that run on across the taps (K = R*S*Cin in order).
template <int MODE>
__host__ __device__ __forceinline__ int count_kb(const TcParams& p) {
    if (MODE == 7) return (p.K + BK / 2 - 1) / (BK / 2);   // 32-bit operands: 32 elements fill a 128-byte row
    if (MODE == 4) return (p.R * p.S * p.Cin + BK - 1) / BK;
    if (MODE == 5) return p.R * ((p.S * p.Cin + BK - 1) / BK);   // filter rows in 64-element pieces (TcParams::a_rowtaps)
    if (MODE == 2) return p.R * p.S * ((p.Cin + BK - 1) / BK);
    const int bk = p.in_dt == FC_F8E4M3 ? 2 * BK : BK;
    return (p.K + bk - 1) / bk;
}

template <int BN, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmSA,
               const __grid_constant__ CUtensorMap tmSB, const TcParams p) {
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    // the same offset in both CTAs of the pair: the MMA addresses the peer's tiles by this CTA's descriptors
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    constexpr int ring_bytes = C::kStages * C::kStageBytes;   // operand stages: A and B side by side per stage
    float* svec_all = reinterpret_cast<float*>(smem + ring_bytes);
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + ring_bytes + C::kVecBytes);
    float2* xchg = reinterpret_cast<float2*>(smem + ring_bytes + C::kVecBytes + C::kCtrlBytes);
    float* pool_stage = reinterpret_cast<float*>(smem + ring_bytes + C::kVecBytes + C::kCtrlBytes + C::kXchgBytes);
    constexpr bool kMx = MODE == 6;
    uint8_t* scale_ring = smem + ring_bytes + C::kVecBytes + C::kCtrlBytes + C::kXchgBytes + C::kPoolBytes;   // mode 6: [stage][A tile 512 B | B tile 512 B]
    volatile int* abort_flag = &ctrl->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = ptx::cluster_ctarank();
    const bool leader = cta_rank == 0;
    const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
    // 4: the convolution with eight filter taps per k-block (TcParams::a_packed); 5: with a filter row per k-block
    // (TcParams::a_rowtaps).  Instantiations of their own: as run-time branches of mode 2's producer either of them
    // cost the ordinary convolution 2 - 10 %.
    constexpr bool kConv = MODE == 2 || MODE == 4 || MODE == 5;
    // rows of the output that a CTA's tile stands for: all 128, or (convolution + max-pool in whole row pairs,
    // TcParams::m_rows) the first m_rows of them: the tile still loads and multiplies 128 positions, the last ones
    // belong to the next tile and are dropped here
    const int m_rows = kConv ? p.m_rows : BM;
    const int tiles_m = (p.M + 2 * m_rows - 1) / (2 * m_rows);   // pair-panels of 2 * m_rows rows
    const int tiles_n = (p.N + BN - 1) / BN;
    const int total_tiles = tiles_m * tiles_n;
    const int kb_per_tap = kConv ? (p.Cin + BK - 1) / BK : 1;
    const bool f8 = !kConv && (kMx || p.in_dt == FC_F8E4M3);
    const int bk = MODE == 7 ? BK / 2 : (f8 ? 2 * BK : BK);   // K elements per k-block: 128 bytes of a row
    const int num_kb = count_kb<MODE>(p);
    const int total_units = p.split > 1 ? p.split_from + (total_tiles - p.split_from) * p.split : total_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->full[s]), 1);    // the leader's arrive.expect_tx for both CTAs' bytes
            ptx::mbar_init(ptx::smem_u32(&ctrl->empty[s]), 1);   // the leader's commit
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->tfull[b]), 1);   // the leader's commit
            ptx::mbar_init(ptx::smem_u32(&ctrl->tempty[b]), 16); // 8 epilogue warps of each CTA
        }
        ctrl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB);
        if constexpr (kMx) {
            ptx::prefetch_tensormap(&tmSA);
            ptx::prefetch_tensormap(&tmSB);
        }
    }
    // a power of two must be asked for: two 240-column accumulators take 512 like two of 256 (mode 6 puts its scales behind them)
    constexpr int kTmemNeed = C::kTmemCols + (kMx ? 4 + 4 * ((BN + 127) / 128) : 0);
    constexpr int kTmemAlloc = kTmemNeed > 256 ? 512 : 256;
    static_assert(kTmemNeed <= kTmemAlloc, "tensor-memory allocation");
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&ctrl->tmem_base), kTmemAlloc);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync();   // the peer's barriers exist before anything is signalled on them
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    // Launched with programmatic stream serialization: everything above ran while the kernel in front was draining;
    // nothing below touches global memory before that kernel has completed.  (Behind the zero-fill kernel of the
    // convolution only the epilogue warps wait: see there.)
    if (!(kConv && p.after_zero_fill)) asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t hs = 0, hph = 0;   // stage and phase of the operand ring
            bool ok = true;
            long long ppw = 0, ppq = 0, ppt0 = clock64();
            for (int u = cluster_id; u < total_units && ok; u += num_clusters) {
                const Unit w = unit_decode(u, p.split_from, p.split, p.split_kb, num_kb);
                int mb2, nb;
                tile_coords((MODE == 0 || MODE == 6 || MODE == 7 || MODE == 3 || (MODE == 1 && p.two_pass)) ? 0 : 1, p.group_m, w.tile, tiles_m, tiles_n, mb2, nb);   // (the two-pass softmax waits for nobody: free to use the L2-friendly order)
                const int row0 = (mb2 * 2 + (int) cta_rank) * m_rows;      // this CTA's rows of A
                const int bcol0 = nb * BN + (int) cta_rank * (BN / 2);     // this CTA's half of the B tile
                int img = 0, oh = 0, ow = 0;
                if constexpr (kConv) {
                    const int hw = p.OH * p.OW;
                    img = row0 / hw;
                    const int rem = row0 - img * hw;
                    oh = rem / p.OW;
                    ow = rem - oh * p.OW;
                }
                // (mode 2: filter tap and channel slice of the k-block, carried along instead of divided out per block)
                int c0 = 0, tap_r = 0, tap_s = 0, tap_col = 0;
                if constexpr (MODE == 2) {
                    const int tap = w.kb0 / kb_per_tap;
                    c0 = (w.kb0 - tap * kb_per_tap) * BK;
                    tap_r = tap / p.S;
                    tap_s = tap - tap_r * p.S;
                    tap_col = tap * p.Cin;
                } else if constexpr (MODE == 5) {
                    // k-blocks are 64-element pieces of filter rows (one piece where S * Cin <= 64): the S taps of row
                    // r from element c0 on in one copy (tap offset (0, r), channel c0 of the wide "pixel"), the
                    // weights from column r * S * Cin + c0 on
                    const int per_row = (p.S * p.Cin + BK - 1) / BK;
                    tap_r = w.kb0 / per_row;
                    c0 = (w.kb0 - tap_r * per_row) * BK;
                    tap_col = tap_r * p.S * p.Cin + c0;
                }
                for (int kb = w.kb0; kb < w.kb1; ++kb) {
                    const uint32_t s = hs, ph = hph;
                    if (++hs == (uint32_t) C::kStages) { hs = 0; hph ^= 1u; }
                    PROF_T0(ppq);
                    if (!(ok = wait_bar(ptx::smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, p.status))) break;
                    PROF_ADD(ppw, ppq);
                    const uint32_t full = ptx::mapa(ptx::smem_u32(&ctrl->full[s]), 0);   // the leader's barrier
                    const uint32_t sa = ptx::smem_u32(smem + s * C::kStageBytes);
                    // the leader expects the bytes of both CTAs; the peer's copies signal the same barrier.  A
                    // peer copy may land before the expectation is posted: the phase cannot complete before
                    // the leader's arrival, and the peer starts the next phase only after the leader's MMAs
                    // of this one (the commit that frees the stage) are done.
                    if (leader) ptx::mbar_arrive_expect_tx(ptx::smem_u32(&ctrl->full[s]), 2 * (C::kStageBytes + (kMx ? C::kScaleStage : 0)));
                    if constexpr (kMx) {
                        // the scales of this k-block: this CTA's 128 rows of A, the tile's columns of B (one box of one or two tiles)
                        const uint32_t sc = ptx::smem_u32(scale_ring) + s * C::kScaleStage;
                        ptx::tma_load_2d_pair(sc, &tmSA, 0, (mb2 * 2 + (int) cta_rank) * num_kb + kb, full);
                        ptx::tma_load_2d_pair(sc + 512, &tmSB, 0, (nb * num_kb + kb) * ((BN + 127) / 128), full);
                    }
                    if constexpr (MODE == 4) {
                        // eight copies of 128 pixels x 8 channels, each one column of core matrices (2 KB)
                        const int cpt = p.Cin >> 3, chunks = p.R * p.S * cpt;
#pragma unroll 1
                        for (int q = 0; q < 8; ++q) {
                            const int chunk = kb * 8 + q;
                            int c0 = p.Cin, r = 0, sx = 0;     // past the last tap: channels out of range, filled with zeros
                            if (chunk < chunks) {
                                const int tap = chunk / cpt;
                                c0 = (chunk - tap * cpt) * 8;
                                r = tap / p.S;
                                sx = tap - r * p.S;
                            }
                            ptx::tma_load_im2col_4d_pair(sa + q * 2048, &tmA, c0, ow * p.stride - p.pad, oh * p.stride - p.pad, img, (uint16_t) sx, (uint16_t) r, full);
                        }
                        ptx::tma_load_2d_pair(sa + C::kABytes, &tmB, kb * BK, bcol0, full);
                    } else if constexpr (MODE == 2) {
                        ptx::tma_load_im2col_4d_pair(sa, &tmA, c0, ow * p.stride - p.pad, oh * p.stride - p.pad, img, (uint16_t) tap_s, (uint16_t) tap_r, full);
                        ptx::tma_load_2d_pair(sa + C::kABytes, &tmB, tap_col + c0, bcol0, full);
                        c0 += BK;
                        if (c0 >= kb_per_tap * BK) {
                            c0 = 0;
                            tap_col += p.Cin;
                            if (++tap_s == p.S) { tap_s = 0; ++tap_r; }
                        }
                    } else if constexpr (MODE == 5) {
                        ptx::tma_load_im2col_4d_pair(sa, &tmA, c0, ow * p.stride - p.pad, oh * p.stride - p.pad, img, (uint16_t) 0, (uint16_t) tap_r, full);
                        ptx::tma_load_2d_pair(sa + C::kABytes, &tmB, tap_col, bcol0, full);
                        c0 += BK;
                        tap_col += BK;
                        if (c0 >= p.S * p.Cin) {
                            c0 = 0;
                            ++tap_r;
                            tap_col = tap_r * p.S * p.Cin;
                        }
                    } else {
                        ptx::tma_load_2d_pair(sa, &tmA, kb * bk, row0, full);
                        ptx::tma_load_2d_pair(sa + C::kABytes, &tmB, kb * bk, bcol0, full);
                    }
                }
            }
#ifdef FC_PROF
            if (leader && cluster_id < 160) { g_prof[cluster_id][6] = clock64() - ppt0; g_prof[cluster_id][7] = ppw; }
#else
            (void) ppw; (void) ppq; (void) ppt0;
#endif
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (leader && lane == 0) {
            // operand format code: bf16 = 1 and fp16 = 0 under kind::f16, E4M3 = 0 under kind::f8f6f4
            const uint32_t idesc = MODE == 7 ? ptx::idesc_tf32(2 * BM, BN) : ptx::idesc_f16kind_f32(2 * BM, BN, p.in_dt == FC_BF16 ? 1u : 0u);
            uint32_t it = 0, tile_iter = 0;
            bool ok = true;
            long long pw_tempty = 0, pw_full = 0, pw_issue = 0, pt0 = clock64(), pq = 0;
            const unsigned long long pns0 = ptx::globaltimer();
            uint32_t hs = 0, hph = 0;   // stage and phase of the operand ring
            const uint64_t desc0 = ptx::smem_desc_k128(ptx::smem_u32(smem));   // swizzled K-major tile at the first stage
            const uint32_t desc_lo = (uint32_t) desc0, desc_hi = (uint32_t) (desc0 >> 32);
            const uint32_t full0 = ptx::smem_u32(&ctrl->full[0]), empty0 = ptx::smem_u32(&ctrl->empty[0]);
            for (int u = cluster_id; u < total_units && ok; u += num_clusters, ++tile_iter) {
                const Unit w = unit_decode(u, p.split_from, p.split, p.split_kb, num_kb);
                const uint32_t buf = tile_iter & 1u, aph = (tile_iter >> 1) & 1u;
                PROF_T0(pq);
                if (!(ok = wait_bar(ptx::smem_u32(&ctrl->tempty[buf]), aph ^ 1u, abort_flag, p.status))) break;
                PROF_ADD(pw_tempty, pq);
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                // This thread's own instruction stream sets the pace of the main loop: per k-block a wait, four MMA
                // issues and a commit leave little of the 512 cycles the tensor pipe needs for them (measured: sixteen
                // more dependent instructions per k-block cost forty cycles each time).  So whole rounds of the stage
                // ring run unrolled, with barrier addresses and descriptor offsets as constants; the k-blocks in front
                // of a round boundary and behind the last whole round take the same body with a run-time stage.
                auto kblock = [&](uint32_t s, uint32_t ph, uint32_t acc0) -> bool {
                    PROF_T0(pq);
                    if (!wait_bar(full0 + 8u * s, ph, abort_flag, p.status)) return false;
                    PROF_ADD(pw_full, pq);
                    ptx::tc_fence_after();
                    PROF_T0(pq);
                    if constexpr (MODE == 4) {
                        // A without swizzle: 2 KB between the core matrices of neighbouring 8-channel chunks, 128
                        // bytes between 8-pixel groups; one MMA takes two chunks
                        const uint64_t dp = ptx::smem_desc_k_plain(ptx::smem_u32(smem) + s * C::kStageBytes, 2048, 128);
                        const uint64_t db = desc0 + (uint64_t) (s * (C::kStageBytes >> 4) + (C::kABytes >> 4));
                        ptx::tc_mma_f16_pair(d_tmem, dp, db, idesc, acc0);
#pragma unroll
                        for (int k = 1; k < BK / 16; ++k)
                            ptx::tc_mma_f16_pair(d_tmem, dp + (uint64_t) (k * (4096 >> 4)), db + 2 * k, idesc, 1u);
                    } else if constexpr (kMx) {
                        // scales into tensor memory (the copies and the MMAs run in the order they are issued), then four
                        // MMAs of 32 elements along K, MMA j with byte j of the scale columns
                        const uint32_t sc = ptx::smem_u32(scale_ring) + s * C::kScaleStage;
                        const uint32_t t_sfa = tmem_base + 2 * BN, t_sfb = t_sfa + 4;
                        ptx::tc_cp_32x128b_pair(t_sfa, ptx::smem_desc_k_plain(sc, 16, 128));
#pragma unroll
                        for (int t = 0; t < (BN + 127) / 128; ++t)
                            ptx::tc_cp_32x128b_pair(t_sfb + 4 * t, ptx::smem_desc_k_plain(sc + 512 + 512 * t, 16, 128));
                        const uint32_t a_lo = desc_lo + s * (uint32_t) (C::kStageBytes >> 4);
                        const uint32_t b_lo = a_lo + (uint32_t) (C::kABytes >> 4);
                        ptx::tc_mma_mxf8_pair_lh(d_tmem, a_lo, b_lo, desc_hi, ptx::idesc_mxf8_e4m3(2 * BM, BN, 0, 0), t_sfa, t_sfb, acc0);
#pragma unroll
                        for (int k = 1; k < 4; ++k)
                            ptx::tc_mma_mxf8_pair_lh(d_tmem, a_lo + 2 * k, b_lo + 2 * k, desc_hi, ptx::idesc_mxf8_e4m3(2 * BM, BN, (uint32_t) k, (uint32_t) k), t_sfa, t_sfb, 1u);
                    } else if constexpr (MODE == 7) {
                        const uint32_t a_lo = desc_lo + s * (uint32_t) (C::kStageBytes >> 4);
                        const uint32_t b_lo = a_lo + (uint32_t) (C::kABytes >> 4);
                        ptx::tc_mma_tf32_pair_lh(d_tmem, a_lo, b_lo, desc_hi, idesc, acc0);
#pragma unroll
                        for (int k = 1; k < 4; ++k)  // 8 values of 32 bits = 32 bytes per MMA along K -> +2 in 16-byte units
                            ptx::tc_mma_tf32_pair_lh(d_tmem, a_lo + 2 * k, b_lo + 2 * k, desc_hi, idesc, 1u);
                    } else {
                        const uint32_t a_lo = desc_lo + s * (uint32_t) (C::kStageBytes >> 4);   // stage s, A tile; B follows kABytes further on
                        const uint32_t b_lo = a_lo + (uint32_t) (C::kABytes >> 4);
                        if (f8) {
                            ptx::tc_mma_f8_pair_lh(d_tmem, a_lo, b_lo, desc_hi, idesc, acc0);
#pragma unroll
                            for (int k = 1; k < 4; ++k)  // 32 E4M3 values = 32 bytes per MMA along K -> +2 in 16-byte units
                                ptx::tc_mma_f8_pair_lh(d_tmem, a_lo + 2 * k, b_lo + 2 * k, desc_hi, idesc, 1u);
                        } else {
                            ptx::tc_mma_f16_pair_lh(d_tmem, a_lo, b_lo, desc_hi, idesc, acc0);
#pragma unroll
                            for (int k = 1; k < BK / 16; ++k)  // 16 bf16 = 32 bytes per MMA along K -> +2 in 16-byte units
                                ptx::tc_mma_f16_pair_lh(d_tmem, a_lo + 2 * k, b_lo + 2 * k, desc_hi, idesc, 1u);
                        }
                    }
                    ptx::tc_commit_pair(empty0 + 8u * s, 3);     // frees the stage in both CTAs
                    PROF_ADD(pw_issue, pq);
                    return true;
                };
                int kb = w.kb0;
                uint32_t acc = 0;   // the unit's first MMA overwrites the accumulator
                for (; ok && kb < w.kb1 && hs != 0; ++kb, ++it) {   // up to the next round boundary
                    ok = kblock(hs, hph, acc);
                    acc = 1;
                    if (++hs == (uint32_t) C::kStages) { hs = 0; hph ^= 1u; }
                }
                for (; ok && kb + C::kStages <= w.kb1; kb += C::kStages, it += C::kStages) {   // whole rounds
#pragma unroll
                    for (int s = 0; s < C::kStages; ++s)
                        if (ok) ok = kblock((uint32_t) s, hph, s == 0 ? acc : 1u);
                    acc = 1;
                    hph ^= 1u;
                }
                for (; ok && kb < w.kb1; ++kb, ++it) {   // the rest of the unit
                    ok = kblock(hs, hph, acc);
                    acc = 1;
                    if (++hs == (uint32_t) C::kStages) { hs = 0; hph ^= 1u; }
                }
                if (ok) ptx::tc_commit_pair(ptx::smem_u32(&ctrl->tfull[buf]), 3);   // accumulators ready in both CTAs
            }
#ifdef FC_PROF
            if (cluster_id < 160) {
                g_prof[cluster_id][0] = clock64() - pt0; g_prof[cluster_id][1] = pw_tempty; g_prof[cluster_id][2] = 0; g_prof[cluster_id][3] = pw_full;
                g_prof[cluster_id][4] = it; g_prof[cluster_id][5] = pw_issue; g_prof[cluster_id][8] = (long long) (ptx::globaltimer() - pns0);
            }
#else
            (void) pns0; (void) pt0; (void) pw_tempty; (void) pw_full; (void) pw_issue; (void) pq;
#endif
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps (both CTAs)
        const int lane_grp = warp & 3;
        const int half = (warp - 2) >> 2;  // which half of the tile's columns this warp handles
        const int row = lane_grp * 32 + lane;
        const int et = threadIdx.x - 64;   // 0..255
        const uint32_t lane_addr = (uint32_t) (lane_grp * 32) << 16;
        const bool precise = false;   // tanh.approx GELU is accurate to 6e-6 on sm_100a (see gelu_tanh)
        const bool out_vec = (reinterpret_cast<uintptr_t>(p.out) & 15) == 0 && (p.N & 7) == 0;
        const uint32_t tempty_leader = ptx::mapa(ptx::smem_u32(&ctrl->tempty[0]), 0);
        // debug build: the main output's extent for the address checks of the stores
        const DbgOut dbg_out = {kConv ? 0 : (long long) p.M * p.N * (p.out_dt == FC_F32 ? 4 : 2) - p.dbg_trim, p.status};
        const long long dbg_stats_bytes = (long long) p.M * tiles_n * 8 * (MODE == 1 && p.two_pass ? 2 : 1);
        (void) dbg_stats_bytes;
        if constexpr (kConv) {
            // the pooled output is zeroed by the kernel in front, which this one was allowed to overtake: only
            // these warps, the ones that update the output, wait for it (a no-op under an ordinary launch)
            if (p.after_zero_fill) asm volatile("griddepcontrol.wait;" ::: "memory");
        }
        uint32_t tile_iter = 0;
        int staged_nb0 = -1, staged_nb1 = -1;   // column tile whose vectors each staging buffer holds
        for (int u = cluster_id; u < total_units; u += num_clusters, ++tile_iter) {
            const Unit w = unit_decode(u, p.split_from, p.split, p.split_kb, num_kb);
            int mb2, nb;
            tile_coords((MODE == 0 || MODE == 6 || MODE == 7 || MODE == 3 || (MODE == 1 && p.two_pass)) ? 0 : 1, p.group_m, w.tile, tiles_m, tiles_n, mb2, nb);   // (the two-pass softmax waits for nobody: free to use the L2-friendly order)
            const int mb = mb2 * 2 + (int) cta_rank;    // 128-row panel of this CTA
            const uint32_t buf = tile_iter & 1u, aph = (tile_iter >> 1) & 1u;
            const int n_tile = nb * BN;
            float* svec = svec_all + buf * (kMaxVecSlots * BN);
            EPI_MARK(0);
            // stage this tile's slices of the per-column vectors (fp32) before the accumulator wait (not again when the
            // buffer holds this column tile's already: every tile of a convolution narrower than a tile, 700 cycles of
            // global-load latency per tile that an epilogue-bound layer cannot hide)
            if ((buf ? staged_nb1 : staged_nb0) != nb) {
                if (buf) staged_nb1 = nb;
                else staged_nb0 = nb;
                int slot = 0;
                for (int i = 0; i < p.ops.n && slot < kMaxVecSlots; ++i) {
                    const DevOp& op = p.ops.op[i];
                    const int nvec = op.kind == FC_OP_BIAS_N ? 1 : (op.kind == FC_OP_AFFINE_N ? 2 : 0);
                    for (int k = 0; k < nvec && slot < kMaxVecSlots; ++k, ++slot)
                        for (int c = et; c < BN; c += kEpiThreads)
                            svec[slot * BN + c] = n_tile + c < p.N ? load_scalar(k ? op.p1 : op.p0, k ? op.dt1 : op.dt0, n_tile + c) : 0.0f;
                }
            }
            // one thread waits for the accumulator; its verdict reaches all four warps through shared
            // memory and a named barrier, so that they leave the loop together or not at all
            if (et == 0) ctrl->epi_ok[buf] = wait_bar(ptx::smem_u32(&ctrl->tfull[buf]), aph, abort_flag, p.status);
            ptx::bar_sync(2, kEpiThreads);
            if (!*(volatile int*) &ctrl->epi_ok[buf]) break;
            ptx::tc_fence_after();
            EPI_MARK(1);
            constexpr int kChunks = C::kColHalf / 16;  // 16-column chunks per thread (half a tile row; 240-column tiles: 8 and 7)
            const int n_chunks = BN == 240 && half == 1 ? kChunks - 1 : kChunks;   // chunks of this half that belong to the tile
            const int col_half = half * C::kColHalf;
            const int n_lim = min(p.N, n_tile + BN);   // first column that is not this tile's
            const uint32_t tacc = tmem_base + buf * BN + col_half + lane_addr;
            // (rows of the tile behind m_rows: no row of the output, which `m >= M` says everywhere below)
            const long long m = row < m_rows ? (long long) mb * m_rows + row : (long long) p.M;
            const int n_half = n_tile + col_half;
            // hands the accumulator buffer back to the leader's MMA thread
            auto release_buf = [&]() {
                ptx::tc_fence_before();
                __syncwarp();
                // relaxed: every lane's accumulator reads are complete (tcgen05.wait::ld) before the __syncwarp above,
                // and a release here would hold the warp until its global stores of this tile have drained
                if (lane == 0) ptx::mbar_arrive_cluster_relaxed(tempty_leader + buf * 8);
            };

            if (w.nsl > 1) {
                // Slice of a split tile.  Scratch layout per (slice, CTA): [warp 8][chunk][quad 4][lane 32] float4,
                // so that every warp instruction moves 512 contiguous bytes.
                constexpr size_t kSliceF4 = (size_t) BM * 2 * C::kColHalf / 4;
                const int ws = warp - 2;
                unsigned int* cnt = &p.split_counters[(w.v0 / w.nsl) * 2 + (int) cta_rank];
                // a warp none of whose 32 rows exists (a short last panel: 16 rows of 256; rows behind m_rows) parks and merges nothing
                // (warp-uniform: the loops below issue warp-wide accumulator loads)
                const bool live = lane_grp * 32 < m_rows && (long long) mb * m_rows + lane_grp * 32 < p.M;
                if (w.slice != w.nsl - 1) {
                    float4* mine = p.split_ws + ((size_t) (w.v0 + w.slice) * 2 + cta_rank) * kSliceF4 + (size_t) ws * kChunks * 128 + lane;
#pragma unroll 1
                    for (int c = 0; live && c < kChunks; c += 2) {
                        uint32_t ra[16], rb[16];
                        ptx::tmem_ld_32x16_async(tacc + c * 16, ra);
                        ptx::tmem_ld_32x16_async(tacc + (c + 1) * 16, rb);
                        ptx::tmem_wait_ld(ra);
                        ptx::tmem_wait_ld(rb);
                        if (!FC_DBG_IN(mine + c * 4 * 32, 2 * 4 * 32 * 16 - 31 * 16, p.split_ws, (long long) kTcSplitUnits * 2 * BM * 256 * 4, p.status, kSiteSplitPark)) continue;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            __stcg(mine + (c * 4 + j) * 32, make_float4(__uint_as_float(ra[4 * j]), __uint_as_float(ra[4 * j + 1]), __uint_as_float(ra[4 * j + 2]), __uint_as_float(ra[4 * j + 3])));
                            __stcg(mine + ((c + 1) * 4 + j) * 32, make_float4(__uint_as_float(rb[4 * j]), __uint_as_float(rb[4 * j + 1]), __uint_as_float(rb[4 * j + 2]), __uint_as_float(rb[4 * j + 3])));
                        }
                    }
                    __threadfence();
                    ptx::bar_sync(1, kEpiThreads);
                    if (et == 0) ptx::red_release_gpu_add(cnt, 1u);
                    release_buf();
                    continue;
                }
                // the merging slice: wait (bounded) until the others have parked their rows
                if (et == 0) {
                    const unsigned long long t0 = ptx::globaltimer();
                    unsigned spins = 0;
                    bool ok = true;
                    while (ptx::ld_acquire_gpu(cnt) < (unsigned) (w.nsl - 1 + (MODE == 1 ? 0 : p.expect_extra))) {
                        if ((++spins & 63u) == 0) {
                            if (*abort_flag) { ok = false; break; }
                            if (ptx::globaltimer() - t0 > kWaitLimitNs) {
                                *abort_flag = 1;
                                atomicExch(p.status, kStatusTimeout);
                                ok = false;
                                break;
                            }
                        }
                    }
                    if (ok) *cnt = 0u;   // nobody else touches it in this launch: the next launch finds zero
                    ctrl->merge_ok = ok;
                    __threadfence();
                }
                ptx::bar_sync(1, kEpiThreads);
                if (!*(volatile int*) &ctrl->merge_ok) break;
                // add the other slices' rows into the accumulator, four chunks of loads in flight
#pragma unroll 1
                for (int c0 = 0; live && c0 < kChunks; c0 += 4) {
                    float4 acc[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) acc[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                    for (int q = 0; q < w.nsl; ++q) {
                        if (q == w.slice) continue;
                        const float4* src = p.split_ws + ((size_t) (w.v0 + q) * 2 + cta_rank) * kSliceF4 + (size_t) ws * kChunks * 128 + lane + c0 * 128;
                        float4 t[16];
                        if (!FC_DBG_IN(src, 15 * 32 * 16 + 16, p.split_ws, (long long) kTcSplitUnits * 2 * BM * 256 * 4, p.status, kSiteSplitMerge)) continue;
#pragma unroll
                        for (int i = 0; i < 16; ++i) t[i] = __ldcg(src + i * 32);
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            acc[i].x += t[i].x; acc[i].y += t[i].y; acc[i].z += t[i].z; acc[i].w += t[i].w;
                        }
                    }
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t r[16];
                        ptx::tmem_ld_32x16_async(tacc + (c0 + cc) * 16, r);
                        ptx::tmem_wait_ld(r);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            r[4 * j] = __float_as_uint(__uint_as_float(r[4 * j]) + acc[cc * 4 + j].x);
                            r[4 * j + 1] = __float_as_uint(__uint_as_float(r[4 * j + 1]) + acc[cc * 4 + j].y);
                            r[4 * j + 2] = __float_as_uint(__uint_as_float(r[4 * j + 2]) + acc[cc * 4 + j].z);
                            r[4 * j + 3] = __float_as_uint(__uint_as_float(r[4 * j + 3]) + acc[cc * 4 + j].w);
                        }
                        if (c0 + cc < n_chunks) ptx::tmem_st_32x16(tacc + (c0 + cc) * 16, r);
                    }
                }
                ptx::tmem_wait_st();
            }

            if constexpr (MODE == 0 || MODE == 6 || MODE == 7) {
                // one chunk at a time, one copy of the code: load, wait, ops, store (keeping the next load in flight
                // and two copies of this body was no faster; see tmem_sweep)
#pragma unroll 1
                for (int c = 0; c < n_chunks; ++c) {
                    const int n0 = n_half + c * 16;
                    if (n0 >= n_lim) break;
                    uint32_t r[16];
                    ptx::tmem_ld_32x16_async(tacc + c * 16, r);
                    ptx::tmem_wait_ld(r);
                    float v[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
                    if (m < p.M) {
                        if (precise) apply_ops16<true>(v, p.ops, svec, BN, col_half + c * 16, m, n0, p.N, p.N);
                        else apply_ops16<false>(v, p.ops, svec, BN, col_half + c * 16, m, n0, p.N, p.N);
                    }
                    if (!out_vec) {
                        // rows off 16-byte boundaries: the warp stores its 32 x 16 block together
                        store16_rows(p.out, p.out_dt, pool_stage + (warp - 2) * (32 * 17), v, m - lane, p.M, n0, p.N, lane, dbg_out);
                    } else if (m < p.M) {
                        store16(p.out, p.out_dt, out_vec, v, m, n0, p.N, dbg_out);
                    }
                }
            } else if constexpr (MODE == 3) {
                // ops, optional store, and a running reduction of the row slice: (max, sum of exponentials) in
                // the log2 domain for logsumexp, a plain sum or maximum otherwise.  The tile that publishes
                // last for its row panel merges all slices, so nobody waits for anybody.
                const int rk = p.red_kind;
                float run_m = -CUDART_INF_F, run_s = 0.0f;
#pragma unroll 1
                for (int c = 0; c < kChunks; ++c) {
                    uint32_t r[16];
                    ptx::tmem_ld_32x16_async(tacc + c * 16, r);
                    ptx::tmem_wait_ld(r);
                    const int n0 = n_half + c * 16;
                    if (p.out && !out_vec && n0 < n_lim) {
                        // rows off 16-byte boundaries: every lane takes part in the store of the warp's block
                        float v[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
                        if (m < p.M) apply_ops16<false>(v, p.ops, svec, BN, col_half + c * 16, m, n0, p.N, p.N);
                        store16_rows(p.out, p.out_dt, pool_stage + (warp - 2) * (32 * 17), v, m - lane, p.M, n0, p.N, lane, dbg_out);
                    }
                    if (m < p.M && n0 < n_lim) {
                        float v[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
                        apply_ops16<false>(v, p.ops, svec, BN, col_half + c * 16, m, n0, p.N, p.N);
                        if (p.out && out_vec) store16(p.out, p.out_dt, out_vec, v, m, n0, p.N, dbg_out);
                        if (rk == FC_RED_ROW_LOGSUMEXP || rk == FC_RED_ROW_MAX) {
                            float cm = -CUDART_INF_F;
#pragma unroll
                            for (int j = 0; j < 16; ++j) cm = n0 + j < p.N ? fmaxf(cm, v[j]) : cm;
                            if (rk == FC_RED_ROW_MAX) {
                                run_m = fmaxf(run_m, cm);
                            } else {
                                const float nm = fmaxf(run_m, cm * kLog2e);
                                // only -inf so far (an additive mask): exponents against 0, so that they stay -inf
                                const float base = nm == -CUDART_INF_F ? 0.0f : nm;
                                float cs = 0.0f;
#pragma unroll
                                for (int j = 0; j < 16; ++j) cs += n0 + j < p.N ? exp2_fast(fmaf(v[j], kLog2e, -base)) : 0.0f;
                                run_s = fmaf(run_s, exp2_fast(run_m - base), cs);
                                run_m = nm;
                            }
                        } else {
                            float cs = 0.0f;
#pragma unroll
                            for (int j = 0; j < 16; ++j) cs += n0 + j < p.N ? v[j] : 0.0f;
                            run_s += cs;
                        }
                    }
                }
                // merge of two partial results of one row, by kind
                auto merge = [rk](float am, float as, float bm, float bs) {
                    if (rk == FC_RED_ROW_LOGSUMEXP) {
                        const float nm = fmaxf(am, bm);
                        const float sa = am == -CUDART_INF_F ? 0.0f : as * exp2_fast(am - nm);
                        const float sb = bm == -CUDART_INF_F ? 0.0f : bs * exp2_fast(bm - nm);
                        return make_float2(nm, sa + sb);
                    }
                    return make_float2(fmaxf(am, bm), as + bs);
                };
                if (half == 1) xchg[row] = make_float2(run_m, run_s);
                ptx::bar_sync(1, kEpiThreads);
                if (half == 0 && m < p.M) {
                    const float2 o = xchg[row];
                    if (FC_DBG_IN(&p.stats[(long long) nb * p.M + m], 8, p.stats, dbg_stats_bytes, p.status, kSiteStats))
                        __stcg(&p.stats[(long long) nb * p.M + m], merge(run_m, run_s, o.x, o.y));
                }
                __threadfence();
                ptx::bar_sync(1, kEpiThreads);
                if (et == 0) {
                    const bool last = ptx::atom_acq_rel_gpu_add(&p.counters[mb], 1u) == (unsigned) tiles_n - 1u;
                    if (last) p.counters[mb] = 0u;   // left at zero for the next launch
                    ctrl->last = last;
                    __threadfence();
                }
                ptx::bar_sync(1, kEpiThreads);
                if (*(volatile int*) &ctrl->last && half == 0 && m < p.M) {
                    float2 a = make_float2(-CUDART_INF_F, 0.0f);
                    for (int j = 0; j < tiles_n; ++j) {
                        const float2 st = __ldcg(&p.stats[(long long) j * p.M + m]);
                        a = merge(a.x, a.y, st.x, st.y);
                    }
                    if (FC_DBG_IN(&p.red[m], 4, p.red, (long long) p.M * 4, p.status, kSiteRowResult))
                    p.red[m] = rk == FC_RED_ROW_LOGSUMEXP ? (a.x + log2f(a.y)) * kLn2
                             : rk == FC_RED_ROW_MAX ? a.x
                             : rk == FC_RED_ROW_MEAN ? a.y / (float) p.N : a.y;
                }
            } else if constexpr (MODE == 1) {
                // sweep A: maximum of this thread's half row of the tile (ops applied, written back in place
                // when the list is not empty, so that the later sweeps read finished logits)
                const bool has_ops = p.ops.n > 0;
                float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
                tmem_sweep<kChunks>(tacc, n_chunks, [&](int c, uint32_t (&r)[16]) {
                    const int n0 = n_half + c * 16;
                    if (has_ops) {
                        float v[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
                        if (m < p.M && n0 < n_lim) apply_ops16<false>(v, p.ops, svec, BN, col_half + c * 16, m, n0, p.N, p.N);
#pragma unroll
                        for (int j = 0; j < 16; ++j) r[j] = __float_as_uint(v[j]);
                        ptx::tmem_st_32x16(tacc + c * 16, r);
                    }
                    if (m < p.M && n0 + 16 <= n_lim) {
                        // (four chains instead of one: the sweep's time was the latency of 128 dependent maxima)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            mx4[0] = fmaxf(mx4[0], __uint_as_float(r[4 * j]));
                            mx4[1] = fmaxf(mx4[1], __uint_as_float(r[4 * j + 1]));
                            mx4[2] = fmaxf(mx4[2], __uint_as_float(r[4 * j + 2]));
                            mx4[3] = fmaxf(mx4[3], __uint_as_float(r[4 * j + 3]));
                        }
                    } else if (m < p.M && n0 < n_lim) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) mx4[0] = n0 + j < p.N ? fmaxf(mx4[0], __uint_as_float(r[j])) : mx4[0];
                    }
                });
                const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                if (has_ops) ptx::tmem_wait_st();
                EPI_MARK(2);
                if (p.two_pass) {
                    // Two-kernel form: nobody waits for the panel.  One more sweep computes the exponentials against
                    // this half row's own maximum (values in (0, 1]), sums them and stores them at once; the pair
                    // (max, sum) of every (row, tile, half) goes to the workspace and the rescale kernel behind this
                    // one finishes the rows.
                    const float2 l2e = make_float2(kLog2e, kLog2e);
                    const float mbase = mx == -CUDART_INF_F ? 0.0f : mx;   // a half row of -inf only: exponents against 0
                    const float2 moff = make_float2(-mbase * kLog2e, -mbase * kLog2e);
                    float2 acc2 = make_float2(0.0f, 0.0f);
                    const bool ok = *abort_flag == 0;
                    tmem_sweep<kChunks>(tacc, n_chunks, [&](int c, uint32_t (&r)[16]) {
                        const int n0 = n_half + c * 16;
                        if (n0 >= n_lim) return;
                        float v[16];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float2 t = __ffma2_rn(make_float2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1])), l2e, moff);
                            float2 e = make_float2(exp2_fast(t.x), exp2_fast(t.y));
                            if (n0 + 2 * j >= p.N) e.x = 0.0f;
                            if (n0 + 2 * j + 1 >= p.N) e.y = 0.0f;
                            acc2 = __fadd2_rn(acc2, e);
                            v[2 * j] = e.x;
                            v[2 * j + 1] = e.y;
                        }
                        if (!out_vec) {
                            if (__all_sync(0xffffffffu, ok)) store16_rows(p.out, p.out_dt, pool_stage + (warp - 2) * (32 * 17), v, m - lane, p.M, n0, p.N, lane, dbg_out);
                        } else if (m < p.M && ok) {
                            store16(p.out, p.out_dt, out_vec, v, m, n0, p.N, dbg_out);
                        }
                    });
                    if (m < p.M && FC_DBG_IN(&p.stats[(m * tiles_n + nb) * 2 + half], 8, p.stats, dbg_stats_bytes, p.status, kSiteStats))
                        __stcg(&p.stats[(m * tiles_n + nb) * 2 + half], make_float2(mx, acc2.x + acc2.y));
                    release_buf();
                    continue;
                }
                // sweep B: e = 2^((v - max) log2 e), summed, and written back over the logits: the last sweep
                // only rescales, so every element costs one exponential
                float sm = 0.0f;
                {
                    const float2 l2e = make_float2(kLog2e, kLog2e);
                    // a half row of -inf only (an additive mask): exponents against 0, so that they stay -inf
                    const float mbase = mx == -CUDART_INF_F ? 0.0f : mx;
                    const float2 moff = make_float2(-mbase * kLog2e, -mbase * kLog2e);
                    float2 acc2 = make_float2(0.0f, 0.0f);
                    tmem_sweep<kChunks>(tacc, n_chunks, [&](int c, uint32_t (&r)[16]) {
                        const int n0 = n_half + c * 16;
                        if (m < p.M && n0 < n_lim) {
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float2 t = __ffma2_rn(make_float2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1])), l2e, moff);
                                float2 e = make_float2(exp2_fast(t.x), exp2_fast(t.y));
                                if (n0 + 2 * j >= p.N) e.x = 0.0f;
                                if (n0 + 2 * j + 1 >= p.N) e.y = 0.0f;
                                acc2 = __fadd2_rn(acc2, e);
                                r[2 * j] = __float_as_uint(e.x);
                                r[2 * j + 1] = __float_as_uint(e.y);
                            }
                        }
                        ptx::tmem_st_32x16(tacc + c * 16, r);
                    });
                    ptx::tmem_wait_st();
                    sm = acc2.x + acc2.y;
                }
                EPI_MARK(3);
                // the two column halves of a row meet in shared memory; the lower half publishes the tile's pair
                if (half == 1) xchg[row] = make_float2(mx, sm);
                ptx::bar_sync(1, kEpiThreads);
                if (half == 0 && m < p.M) {
                    const float2 o = xchg[row];
                    const MaxSum a = ms_merge(MaxSum{mx, sm}, MaxSum{o.x, o.y});
                    if (FC_DBG_IN(&p.stats[(long long) nb * p.M + m], 8, p.stats, dbg_stats_bytes, p.status, kSiteStats))
                        __stcg(&p.stats[(long long) nb * p.M + m], make_float2(a.m, a.s));
                }
                // (no fence per thread: the barrier orders the stores above before the one release below, which is
                // cumulative at device scope)
                ptx::bar_sync(1, kEpiThreads);
                // one thread announces the tile and waits (bounded) for the panel's other tiles
                if (et == 0) {
                    ptx::red_release_gpu_add(&p.counters[mb], 1u);
                    const unsigned long long t0 = ptx::globaltimer();
                    unsigned spins = 0;
                    while (ptx::ld_acquire_gpu(&p.counters[mb]) < (unsigned) (tiles_n + p.expect_extra)) {
                        if ((++spins & 63u) == 0) {
                            if (*abort_flag) break;
                            if (ptx::globaltimer() - t0 > kWaitLimitNs) {
                                *abort_flag = 1;
                                atomicExch(p.status, kStatusTimeout);
                                break;
                            }
                        }
                    }
                }
                ptx::bar_sync(1, kEpiThreads);
                EPI_MARK(4);
                const bool store = *abort_flag == 0;
                // Departure count of the panel: asked for here, read after the last sweep, so that its round trip is off
                // the path.  Relaxed (an acquire would hold back the loads below): this tile's last poll of the arrival
                // counter has returned, and whoever reads tiles_n - 1 here resets the counters only after that.
                unsigned departed_before = 0u;
                if (et == 0 && store) departed_before = ptx::atom_relaxed_gpu_add(&p.departed[mb], 1u);
                // The panel's pairs (max, sum) of this row: each column half of the tile merges one half of them, kBatch loads
                // in flight (first the maximum, then the sum of the rescaled partial sums: independent exponentials
                // instead of a chain of merges), and the two halves meet in shared memory.
                MaxSum a = ms_identity();
                if (m < p.M && store) {
                    constexpr int kBatch = 16;
                    const int j_mid = (tiles_n + 1) >> 1;
                    const int j_begin = half == 0 ? 0 : j_mid, j_end = half == 0 ? j_mid : tiles_n;
                    const float2* scol = p.stats + m;   // tile-major: a warp's 32 rows of one tile are 256 consecutive bytes
                    for (int j0 = j_begin; j0 < j_end; j0 += kBatch) {
                        float2 st[kBatch];
#pragma unroll
                        for (int q = 0; q < kBatch; ++q) st[q] = j0 + q < j_end ? __ldcg(scol + (long long) (j0 + q) * p.M) : make_float2(-CUDART_INF_F, 0.0f);
                        float bm = st[0].x;
#pragma unroll
                        for (int q = 1; q < kBatch; ++q) bm = fmaxf(bm, st[q].x);
                        const float base = bm == -CUDART_INF_F ? 0.0f : bm;   // -inf only (an additive mask): the sums are zero
                        float bs = 0.0f;
#pragma unroll
                        for (int q = 0; q < kBatch; ++q) bs = fmaf(st[q].y, exp2_fast((st[q].x - base) * kLog2e), bs);
                        a = ms_merge(a, MaxSum{bm, bs});
                    }
                }
                xchg[half * BM + row] = make_float2(a.m, a.s);
                ptx::bar_sync(1, kEpiThreads);
                {
                    const float2 o = xchg[(half ^ 1) * BM + row];
                    a = ms_merge(a, MaxSum{o.x, o.y});
                }
                const float row_m = a.m, row_s = a.s;
                EPI_MARK(6);
                // last sweep: p = e * 2^((max_half - max_row) log2 e) / sum_row, one factor per thread
                const float fac = m < p.M && store && mx != -CUDART_INF_F ? exp2_fast((mx - row_m) * kLog2e) / row_s : 0.0f;   // (a half row of -inf only holds zeros)
                const float2 fac2 = make_float2(fac, fac);
                tmem_sweep<kChunks>(tacc, n_chunks, [&](int c, uint32_t (&r)[16]) {
                    const int n0 = n_half + c * 16;
                    if (!out_vec && n0 < n_lim && __all_sync(0xffffffffu, store)) {
                        // rows off 16-byte boundaries: the warp stores its 32 x 16 block together
                        float v[16];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float2 t = __fmul2_rn(make_float2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1])), fac2);
                            v[2 * j] = t.x;
                            v[2 * j + 1] = t.y;
                        }
                        store16_rows(p.out, p.out_dt, pool_stage + (warp - 2) * (32 * 17), v, m - lane, p.M, n0, p.N, lane, dbg_out);
                    } else if (m < p.M && n0 < n_lim && store && out_vec) {
                        float v[16];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float2 t = __fmul2_rn(make_float2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1])), fac2);
                            v[2 * j] = t.x;
                            v[2 * j + 1] = t.y;
                        }
                        store16(p.out, p.out_dt, out_vec, v, m, n0, p.N, dbg_out);
                    }
                });
                // the tile that has left the panel wait last puts both counters back to zero for the next launch
                // (off the path between the wait and the stores: nothing in this launch reads them again)
                if (et == 0 && store && departed_before == (unsigned) tiles_n - 1u) {
                    p.counters[mb] = 0u;
                    p.departed[mb] = 0u;
                }
            } else if (p.pool == 1) {
                // conv + 2x2 max-pool of non-negative values (the op list ends with ReLU, the output starts at
                // zero): every pixel that lies in a window takes part in an unsigned atomic maximum on the fp32
                // bit pattern.  Horizontal neighbours are merged by a shuffle first; the values then go through
                // shared memory so that one instruction updates 16 consecutive channels of two windows.
                const int hw = p.OH * p.OW, PH = p.OH >> 1, PW = p.OW >> 1;
                long long dst = 0;
                bool merge = false, emit = false;
                if (m < p.M) {
                    const int img = (int) (m / hw);
                    const int rem = (int) (m - (long long) img * hw);
                    const int oh = rem / p.OW, ow = rem - oh * p.OW;
                    if ((oh >> 1) < PH && (ow >> 1) < PW) {
                        dst = (((long long) img * PH + (oh >> 1)) * PW + (ow >> 1)) * p.N;
                        const bool even = (ow & 1) == 0;
                        merge = even && lane < 31;      // the right neighbour sits in the next lane
                        emit = even || lane == 0;       // an odd pixel is covered by its left neighbour, if this warp has it
                    }
                }
                // Emission slots: in slot k lanes 0-15 serve the (2k)-th emitting pixel of this warp and lanes
                // 16-31 the (2k+1)-th, one channel per lane.  Which pixel that is, whether its right neighbour is
                // merged in, and the window it updates do not depend on the channel chunk: found once per tile.
                const unsigned emit_mask = __ballot_sync(0xffffffffu, emit);
                const unsigned merge_mask = __ballot_sync(0xffffffffu, merge);
                constexpr int kSlots = 9;                  // at most 17 emitters: 16 even pixels and an odd one in lane 0
                const int n_slots = (__popc(emit_mask) + 1) >> 1;
                const int win = (int) (dst / p.N);         // window index, below 2^31 like the pixel index
                int slot_win[kSlots];
                unsigned long long slot_src = 0;           // 7 bits per slot: source lane, merge flag, valid flag
#pragma unroll
                for (int k = 0; k < kSlots; ++k) {
                    const unsigned src = __fns(emit_mask, 0, 2 * k + (lane >> 4) + 1);   // 0xffffffff: no such pixel
                    const bool ok = src < 32u;
                    slot_win[k] = __shfl_sync(0xffffffffu, win, ok ? (int) src : 0);
                    const unsigned code = ok ? (src | ((merge_mask >> src & 1u) << 5) | 64u) : 0u;
                    slot_src |= (unsigned long long) code << (7 * k);
                }
                float* stage = pool_stage + (warp - 2) * (32 * 17);
                unsigned int* out_u = (unsigned int*) p.out;
                const int ch = lane & 15;
                tmem_sweep16<kChunks>(tacc, [&](int c, uint32_t (&r)[16]) {
                    const int n0 = n_half + c * 16;
                    if (n0 >= p.N) return;
                    float v[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
                    if (m < p.M) apply_ops16<false>(v, p.ops, svec, BN, col_half + c * 16, m, n0, p.N, p.N);
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (FC_DBG_IN(&stage[lane * 17 + j], 4, pool_stage, (long long) C::kPoolBytes, p.status, kSitePoolStage)) stage[lane * 17 + j] = v[j];
                    __syncwarp();
#pragma unroll
                    for (int k = 0; k < kSlots; ++k) {
                        if (k < n_slots) {
                            const unsigned code = (unsigned) (slot_src >> (7 * k)) & 127u;
                            const int src = code & 31u;
                            if ((code & 64u) && n0 + ch < p.N) {
                                float x = stage[src * 17 + ch];
                                if (code & 32u) x = fmaxf(x, stage[(src + 1) * 17 + ch]);
                                if (FC_DBG_IN(out_u + (long long) slot_win[k] * p.N + n0 + ch, 4, p.out, (long long) p.batch * PH * PW * p.N * 4, p.status, kSitePoolMax))
                                    atomicMax(out_u + (long long) slot_win[k] * p.N + n0 + ch, __float_as_uint(x) & 0x7fffffffu);
                            }
                        }
                    }
                    __syncwarp();
                });
            } else if (p.pool == 2) {
                // conv + 2x2 max-pool of non-negative values for narrow outputs (the op list ends with ReLU, the output starts
                // at zero; chosen by the caller where most windows lie inside one tile: OW <= 32).
                // The 128 positions of this CTA's tile are consecutive in (image, row, column) order, and the four
                // warps of a column half stage their values of a 16-channel chunk in one buffer, position by position.
                // A window whose upper-left position lies at least OW + 1 positions in front of the tile's end has
                // all four of its positions in that buffer: it is finished here and stored.  The other windows meet
                // their second row through an unsigned atomic maximum on the fp32 bit pattern, as before (their
                // positions sit in two tiles).  Which positions emit, what they cover and where they write does not
                // depend on the channel chunk: listed once per tile, so that in every chunk a half-warp serves one
                // entry with one channel per lane (16 consecutive channels per store or atomic).
                const int hw = p.OH * p.OW, PH = p.OH >> 1, PW = p.OW >> 1;
                const int q = lane_grp * 32 + lane;        // this thread's position in the tile
                int* pool_cnt = reinterpret_cast<int*>(xchg) + half * 256;           // [4] emitters per warp, then the entries
                int2* pool_tab = reinterpret_cast<int2*>(pool_cnt + 4);             // up to 65: (position | flags, window)
                int n_emit = 0;
                int my_pos[2] = {-1, -1}, my_win[2] = {0, 0};   // 16-bit output: this quarter warp's windows (position of the upper left, -1: none)
                if (p.pool_whole) {
                    // Tiles of whole row pairs: the tile starts on a row pair and images are whole numbers of pairs, so
                    // the windows are the first PW column pairs of every pair of rows, numbered like the row pairs:
                    // entry e = (pair, column pair) is written down directly, all complete (no search, no divisions
                    // by the image size; keeping the three small quotients in registers across tiles measured slower).
                    const int pair_len = 2 * p.OW, ppt = m_rows / pair_len;
                    const long long pair0 = (long long) mb * ppt;
                    const long long pairs_left = (long long) (p.M / pair_len) - pair0;
                    n_emit = (int) (pairs_left < ppt ? (pairs_left > 0 ? pairs_left : 0) : ppt) * PW;   // at most 32
                    if (p.out_dt != FC_F32) {
                        // 16-bit output: a quarter warp serves entries e and e + 16, which it works out for itself
                        // (no table, no barrier)
#pragma unroll
                        for (int t = 0; t < 2; ++t) {
                            const int e = (q >> 3) + 16 * t;
                            const int pi = e / PW, j = e - pi * PW;
                            my_pos[t] = e < n_emit ? pi * pair_len + 2 * j : -1;
                            my_win[t] = (int) ((pair0 + pi) * PW + j);
                        }
                    } else {
                        if (q < n_emit) {
                            const int pi = q / PW, j = q - pi * PW;
                            pool_tab[q] = make_int2((pi * pair_len + 2 * j) | 128 | 256, (int) ((pair0 + pi) * PW + j));
                        }
                        ptx::bar_sync(3 + half, 128);
                    }
                } else {
                    int win = 0;
                    bool emit = false, right = false, vert = false;
                    if (m < p.M) {
                        const int img = (int) (m / hw);
                        const int rem = (int) (m - (long long) img * hw);
                        const int oh = rem / p.OW, ow = rem - oh * p.OW;
                        if ((oh >> 1) < PH && (ow >> 1) < PW) {
                            win = (img * PH + (oh >> 1)) * PW + (ow >> 1);      // window index, below 2^31 like the position index
                            if ((ow & 1) == 0) {
                                right = q < BM - 1;                             // the right neighbour (same row) is in this tile
                                const bool top = (oh & 1) == 0;
                                vert = top && right && q + p.OW + 1 <= BM - 1;  // and so is the row below
                                // a lower-left position whose window the upper-left one finishes (that one is OW in front)
                                const bool covered = !top && q >= p.OW && q <= BM - 2;
                                emit = !covered;
                            } else {
                                emit = q == 0;                                  // its left neighbour sits in the tile in front
                            }
                        }
                    }
                    const unsigned emask = __ballot_sync(0xffffffffu, emit);
                    if (lane == 0) pool_cnt[lane_grp] = __popc(emask);
                    ptx::bar_sync(3 + half, 128);
                    int before = 0;
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const int cg = pool_cnt[g];
                        before += g < lane_grp ? cg : 0;
                        n_emit += cg;
                    }
                    if (emit) pool_tab[before + __popc(emask & ((1u << lane) - 1u))] = make_int2(q | (right ? 128 : 0) | (vert ? 256 : 0), win);
                    ptx::bar_sync(3 + half, 128);
                }
                EPI_MARK(2);
                float* stage = pool_stage + half * (BM * 17);     // [position][16 channels + 1]
                unsigned int* out_u = (unsigned int*) p.out;
                const int ch = lane & 15, hwid = q >> 4;           // channel of the chunk, half-warp 0..7 of the column half
                const int below = p.OW * 17;
                const bool out16 = p.out_dt != FC_F32;
                // (two 16-bit channels as one word: rows of an even number of channels, the output on a 4-byte boundary)
                const bool pair16 = (p.N & 1) == 0 && (reinterpret_cast<uintptr_t>(p.out) & 3) == 0;
                auto chunk = [&](int c, uint32_t (&r)[16]) {
                    const int n0 = n_half + c * 16;
                    if (n0 >= p.N) return;
                    float v[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
                    if (m < p.M) apply_ops16<false>(v, p.ops, svec, BN, col_half + c * 16, m, n0, p.N, p.N);
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (FC_DBG_IN(&stage[q * 17 + j], 4, pool_stage, (long long) C::kPoolBytes, p.status, kSitePoolStage)) stage[q * 17 + j] = v[j];
                    ptx::bar_sync(3 + half, 128);
                    if (out16) {
                        // 16-bit output (tiles of whole row pairs only: every entry is a complete window): a quarter
                        // warp per entry, two channels per lane, stored as one 32-bit word where the rows allow it.
                        // (The same loop for fp32 outputs, two words per store, gained them 1 - 3 % and cost this form as
                        // much, as a branch in this loop or as a second copy of it: the fp32 form keeps the loop below.)
                        const int c2 = (lane & 7) * 2;
                        if (n0 + c2 < p.N) {
                            const bool both = pair16 || n0 + c2 + 1 < p.N;
#pragma unroll
                            for (int t = 0; t < 2; ++t) {
                                if (my_pos[t] < 0) continue;
                                const float* sp = stage + my_pos[t] * 17 + c2;
                                const float x0 = fabsf(fmaxf(fmaxf(sp[0], sp[17]), fmaxf(sp[below], sp[below + 17])));
                                const float x1 = fabsf(fmaxf(fmaxf(sp[1], sp[18]), fmaxf(sp[below + 1], sp[below + 18])));
                                unsigned short* dst = (unsigned short*) p.out + (long long) my_win[t] * p.N + n0 + c2;
                                if (!FC_DBG_IN(dst, both ? 4 : 2, p.out, (long long) p.batch * PH * PW * p.N * 2, p.status, kSitePoolMax)) continue;
                                const unsigned short h0 = p.out_dt == FC_BF16 ? __bfloat16_as_ushort(__float2bfloat16_rn(x0)) : __half_as_ushort(__float2half_rn(x0));
                                const unsigned short h1 = p.out_dt == FC_BF16 ? __bfloat16_as_ushort(__float2bfloat16_rn(x1)) : __half_as_ushort(__float2half_rn(x1));
                                if (pair16) {
                                    *reinterpret_cast<unsigned int*>(dst) = (unsigned int) h0 | ((unsigned int) h1 << 16);
                                } else {
                                    dst[0] = h0;
                                    if (both) dst[1] = h1;
                                }
                            }
                        }
                    } else if (n0 + ch < p.N) {
                        for (int e = hwid; e < n_emit; e += 8) {
                            const int2 ent = pool_tab[e];
                            const float* sp = stage + (ent.x & 127) * 17 + ch;
                            float x = sp[0];
                            if (ent.x & 128) x = fmaxf(x, sp[17]);
                            unsigned int* dst = out_u + (long long) ent.y * p.N + n0 + ch;
                            if (!FC_DBG_IN(dst, 4, p.out, (long long) p.batch * PH * PW * p.N * 4, p.status, kSitePoolMax)) continue;
                            if (ent.x & 256) {
                                x = fmaxf(x, fmaxf(sp[below], sp[below + 17]));
                                *dst = __float_as_uint(x) & 0x7fffffffu;
                            } else {
                                atomicMax(dst, __float_as_uint(x) & 0x7fffffffu);
                            }
                        }
                    }
                    ptx::bar_sync(3 + half, 128);
                };
                // Two chunks per thread (64-column tiles): both loads at once and a copy of the body for each, 634 against
                // 664 us on 4096 images of 32 x 32 x 8 -> 64.  More chunks: one copy of the body, run again and again
                // (F3 104.4 -> 101.4 us, 64 images of 32 x 32 x 64 -> 128 36.7 -> 33.8).
                if constexpr (kChunks <= 2) tmem_sweep16<kChunks>(tacc, chunk);
                else tmem_sweep<kChunks>(tacc, kChunks, chunk);
            } else {
                // conv + global average pool: channel sums over this warp's 32 pixels
                const int hw = p.OH * p.OW;
                const long long pix_first = (long long) mb * BM + lane_grp * 32;
                const int img_first = (int) (pix_first / hw);
                const long long pix_last = min(pix_first + 31, (long long) p.M - 1);
                const int img_last = pix_last >= pix_first ? (int) (pix_last / hw) : img_first - 1;
                const int my_img = m < p.M ? (int) (m / hw) : -1;
#pragma unroll 1
                for (int c = 0; c < kChunks; c += 2) {
                    uint32_t ra[16], rb[16];
                    ptx::tmem_ld_32x16_async(tacc + c * 16, ra);
                    ptx::tmem_ld_32x16_async(tacc + (c + 1) * 16, rb);
                    ptx::tmem_wait_ld(ra);
                    ptx::tmem_wait_ld(rb);
                    const int n0 = n_half + c * 16;
                    if (n0 >= p.N) continue;
                    float va[16], vb[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) { va[j] = __uint_as_float(ra[j]); vb[j] = __uint_as_float(rb[j]); }
                    if (m < p.M) {
                        apply_ops16<false>(va, p.ops, svec, BN, col_half + c * 16, m, n0, p.N, p.N);
                        apply_ops16<false>(vb, p.ops, svec, BN, col_half + (c + 1) * 16, m, n0 + 16, p.N, p.N);
                    }
                    for (int img = img_first; img <= img_last; ++img) {
                        float w[32];
#pragma unroll
                        for (int j = 0; j < 16; ++j) { w[j] = my_img == img ? va[j] : 0.0f; w[16 + j] = my_img == img ? vb[j] : 0.0f; }
                        const float s = warp_transpose_sum(w, lane);
                        if (n0 + lane < p.N && FC_DBG_IN((float*) p.out + (long long) img * p.N + n0 + lane, 4, p.out, (long long) p.batch * p.N * 4 - p.dbg_trim, p.status, kSitePoolAvg))
                            atomicAdd((float*) p.out + (long long) img * p.N + n0 + lane, s * p.inv_hw);
                    }
                }
            }
            EPI_MARK(5);
            release_buf();
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
        ptx::tmem_dealloc(tmem_base, kTmemAlloc);
    }
}

// per device and instantiation: resident CTA pairs (0 = not asked yet) and whether the shared-memory limit is set
struct LaunchState {
    std::atomic<int> max_clusters[64];
    std::atomic<bool> attr_set[64];
};

template <int BN, int MODE>
cudaError_t launch_one(const TcParams& p, const CUtensorMap* tmA, const CUtensorMap* tmB, int num_sms, cudaStream_t stream,
                       TcPlan* plan, const CUtensorMap* tmSA = nullptr, const CUtensorMap* tmSB = nullptr) {
    static LaunchState state;   // zero-initialised; filled on first use, idempotently, from any thread
    constexpr int kMaxSmem = 232448;   // 227 KB
    constexpr int smem = Cfg<BN>::kSmemBytes + (MODE == 6 ? Cfg<BN>::kScaleBytes : 0);
    static_assert(smem <= kMaxSmem, "shared memory per CTA");
    auto kernel = gemm_tc_kernel<BN, MODE>;
    cudaError_t e = cudaSuccess;
    int dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    const bool known = dev >= 0 && dev < 64;
    if (!known || !state.attr_set[dev].load(std::memory_order_acquire)) {
        if ((e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
        if (known) state.attr_set[dev].store(true, std::memory_order_release);
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // added for the launch itself, not for the occupancy query
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int resident = known ? state.max_clusters[dev].load(std::memory_order_acquire) : 0;
    if (resident == 0) {
        cfg.gridDim = dim3(num_sms & ~1);
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
        if (e != cudaSuccess) return e;
        resident = n > 0 ? n : 1;
        if (known) state.max_clusters[dev].store(resident, std::memory_order_release);
    }
    const int tiles_n = (p.N + BN - 1) / BN;
    const int m_rows = (MODE == 2 || MODE == 4 || MODE == 5) ? p.m_rows : BM;
    const int tiles = ((p.M + 2 * m_rows - 1) / (2 * m_rows)) * tiles_n;
    int max_pairs = resident;
    if (max_pairs > num_sms / 2) max_pairs = num_sms / 2;
    int clusters = max_pairs < tiles ? max_pairs : tiles;
    // (Row softmax: a tile's epilogue waits for the other column tiles of its row panel.  The pair count used to be
    // rounded down to a multiple of the tiles per panel, so that no panel straddled two rounds; with the epilogue's
    // shorter tail that measures no better for 16 - 18 tiles per panel and 8 - 12 % worse where it idles many pairs:
    // 4096 x 5120 x 4096 on 66 of 74 pairs 132 us, on all 74 116 us.)
    TcParams q = p;
    q.split = 1;
    q.split_from = tiles;
    q.split_kb = 0;
    if (p.split_ws) {
        // Tiles left over after the full rounds (all of them, when there are fewer tiles than pairs) are cut
        // along K so that the last round keeps every pair busy.
        const int num_kb = count_kb<MODE>(p);
        const int full = tiles / max_pairs, tail = tiles - full * max_pairs;
        // (row softmax: only when everything fits one round; cutting the last of several rounds would let
        // row panels straddle rounds, which costs more than the split saves)
        if (tail > 0 && !(MODE == 1 && full > 0)) {
            int s = max_pairs / tail;
            if (s > 8) s = 8;
            if (s > num_kb / 4) s = num_kb / 4;
            if (s * tail > kTcSplitUnits) s = kTcSplitUnits / tail;
            // The merging slice gets kExtra k-blocks more than the others (about the time they need to park),
            // so the critical path of the round is its main loop plus the merge.  Measured, parking and
            // merging cost about as much as kMerge k-blocks of main loop: a split must save more than that.
            constexpr int kExtra = 6, kMerge = 24;
            const int park_kb = s >= 2 ? (num_kb - kExtra > s ? (num_kb - kExtra) / s : 1) : num_kb;
            const int merge_kb = num_kb - park_kb * (s - 1);
            const long long plain = (long long) ((tiles + clusters - 1) / clusters) * num_kb;
            const long long cut = (long long) full * num_kb + merge_kb + kMerge;
            if (s >= 2 && cut < plain) {
                q.split = s;
                q.split_from = full * max_pairs;
                q.split_kb = park_kb;
                clusters = full > 0 ? max_pairs : tail * s;
            }
        }
    }
    if (plan) {
        plan->bn = BN;
        plan->tiles = tiles;
        plan->pairs = clusters;
        plan->split = q.split;
        plan->split_tiles = tiles - q.split_from;
        plan->split_kb = q.split_kb;
        plan->num_kb = count_kb<MODE>(p);
    }
    if (!tmA) return cudaSuccess;   // planning only
    cfg.gridDim = dim3(2 * clusters);
    cfg.numAttrs = 2;   // cluster shape + programmatic stream serialization
    {
        char name[64];
        snprintf(name, sizeof(name), "gemm_tc_mode%d_bn%d%s%s%s", MODE == 5 ? 2 : MODE, BN, q.split > 1 ? "_split" : "", MODE == 1 && p.two_pass ? "_two_pass" : "",
                 MODE == 5 ? "_rowtaps" : "");
        note_kernel(name);
    }
    // (the scale-tile maps are read in mode 6 only; the other modes get the operand maps again)
    return cudaLaunchKernelEx(&cfg, kernel, *tmA, *tmB, tmSA ? *tmSA : *tmA, tmSB ? *tmSB : *tmB, q);
}

template <int BN>
cudaError_t launch_bn(const TcParams& p, const CUtensorMap* tmA, const CUtensorMap* tmB, int num_sms, cudaStream_t stream,
                      TcPlan* plan) {
    if constexpr (BN != 64) {   // (64-column tiles: convolutions of at most 64 output channels only)
        switch (p.mode) {
            case 0: return launch_one<BN, 0>(p, tmA, tmB, num_sms, stream, plan);
            case 1: return launch_one<BN, 1>(p, tmA, tmB, num_sms, stream, plan);
            case 3: return launch_one<BN, 3>(p, tmA, tmB, num_sms, stream, plan);
            case 7: return launch_one<BN, 7>(p, tmA, tmB, num_sms, stream, plan);
            default: break;
        }
    }
    // (the convolutions have no 240-column form: their widths are the channel counts, powers of two as a rule)
    if constexpr (BN == 240) return cudaErrorInvalidValue;
    else {
        if (p.mode != 2) return cudaErrorInvalidValue;
        return p.a_packed    ? launch_one<BN, 4>(p, tmA, tmB, num_sms, stream, plan)
             : p.a_rowtaps ? launch_one<BN, 5>(p, tmA, tmB, num_sms, stream, plan)
                           : launch_one<BN, 2>(p, tmA, tmB, num_sms, stream, plan);
    }
}

cudaError_t launch_any(const TcParams& p, const CUtensorMap* tmA, const CUtensorMap* tmB, int bn, int num_sms, cudaStream_t stream,
                       TcPlan* plan) {
    return bn == 256 ? launch_bn<256>(p, tmA, tmB, num_sms, stream, plan)
         : bn == 240 ? launch_bn<240>(p, tmA, tmB, num_sms, stream, plan)
         : bn == 64  ? launch_bn<64>(p, tmA, tmB, num_sms, stream, plan)
                     : launch_bn<128>(p, tmA, tmB, num_sms, stream, plan);
}

}  // namespace

#ifdef FC_PROF
extern "C" void fc_debug_prof(long long* out) { cudaMemcpyFromSymbol(out, g_prof, sizeof(long long) * 160 * 10); }
extern "C" void fc_debug_prof_epi(long long* out) { cudaMemcpyFromSymbol(out, g_prof_epi, sizeof(long long) * 160 * 64); }
extern "C" void fc_debug_prof_clk(long long* out) { cudaMemcpyFromSymbol(out, g_prof_clk, sizeof(long long) * 160 * 64); }
#endif

size_t gemm_tc_smem_bytes(int bn) { return bn == 256 ? Cfg<256>::kSmemBytes : bn == 240 ? Cfg<240>::kSmemBytes : bn == 64 ? Cfg<64>::kSmemBytes : Cfg<128>::kSmemBytes; }

cudaError_t launch_gemm_tc(const TcParams& p, const CUtensorMap& tmA, const CUtensorMap& tmB, int bn, int num_sms,
                           cudaStream_t stream, int* launches) {
    *launches += 1;
    return launch_any(p, &tmA, &tmB, bn, num_sms, stream, nullptr);
}

cudaError_t launch_gemm_tc_mx(const TcParams& p, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmSA,
                              const CUtensorMap& tmSB, int num_sms, cudaStream_t stream, int* launches) {
    *launches += 1;
    return p.N <= 128 ? launch_one<128, 6>(p, &tmA, &tmB, num_sms, stream, nullptr, &tmSA, &tmSB)
                      : launch_one<240, 6>(p, &tmA, &tmB, num_sms, stream, nullptr, &tmSA, &tmSB);
}

cudaError_t plan_gemm_tc(const TcParams& p, int bn, int num_sms, TcPlan* plan) {
    return launch_any(p, nullptr, nullptr, bn, num_sms, nullptr, plan);
}

}  // namespace fc
