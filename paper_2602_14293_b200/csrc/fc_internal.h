// Internal declarations shared by the host planner and the kernels of the fused-chain library.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "fc.h"

namespace fc {

// ---- epilogue op list as the kernels see it (passed by value in kernel parameters) ----
struct DevOp {
    int kind;          // fc_op_kind
    int dt0, dt1;      // fc_dtype of p0 / p1
    float f0, f1;
    const void* p0;    // vector [N] or tensor [M,N]
    const void* p1;    // second vector (AFFINE_N)
};

// When the list has the shape [scale]? [bias | affine]? [relu | gelu]? [scale]? [clamp]? [add tensor]? the
// host also fills `fused`, which the tensor-core epilogues execute as straight packed-fp32x2 code
// instead of interpreting the list (fewer issue slots, less energy next to a power-bound main loop).
struct FusedOps {
    int valid;
    int pre;           // 0 none, 1 bias (vector slot 0), 2 affine (slots 0 and 1)
    int act;           // 0 none, 1 relu, 2 gelu
    int clamp;         // 0 / 1
    int res;           // 0 / 1: add tensor
    int res_dt;
    float pre_scale;   // a SCALE in front of everything (1 if absent): undoing the scaling of 8-bit operands, 1/sqrt(d) in front of a softmax
    float scale;       // post-activation scale (1 if absent)
    float lo, hi;
    const void* res_ptr;
};

struct DevOps {
    int n;
    DevOp op[FC_MAX_OPS];
    FusedOps fused;
};

// Device status word values (also fc_status values).
constexpr int kStatusTimeout = FC_ERR_TIMEOUT;

// Every bounded device-side wait gives up after this many nanoseconds of %globaltimer.
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

// ---- launchers (defined one per .cu file); all enqueue on `stream` and return a cudaError_t ----
struct EwParams {
    int* status;                // device status word (written by the debug build's address checks only)
    long long dbg_trim;         // debug build: bytes by which the checks believe the main output to be shorter (testing)
    const void* x; int x_dt;
    void* y; int y_dt;          // may be null when !store_main
    float* red;                 // row logsumexp out, or null
    long long M, N;
    int reduce;                 // FC_RED_NONE or a row reduction
    DevOps ops;
};
cudaError_t launch_ew_rowreduce(const EwParams& p, int num_sms, cudaStream_t stream, int* launches);

struct GemmF32Params {
    const float* A; const float* B; float* C;
    int M, N, K;
    DevOps ops;
};
cudaError_t launch_gemm_f32(const GemmF32Params& p, cudaStream_t stream, int* launches);
// fp32 operand [rows, K] -> [rows, 3 K] of tf32-representable pieces (see split_tf32_kernel in layout.cu)
cudaError_t launch_split_tf32(const float* x, float* y, long long rows, long long K, bool is_b, bool beside_previous, cudaStream_t stream,
                              int* launches);

// GEMM + linear ops + row sum / mean without a main output, rewritten as out = A u + C (see collapse.cu)
struct CollapseParams {
    const void* A; const void* B; int in_dt;   // [M,K], [N,K], FC_BF16 or FC_F16
    long long M, N, K;
    DevOps ops;                 // BIAS_N, AFFINE_N and SCALE only
    float* out;                 // [M]
    float post;                 // 1 (sum) or 1/N (mean)
    // carved out of the workspace by the launcher
    double* partial; double* cpart; double* cterm; float* u;
};
cudaError_t launch_collapse(const CollapseParams& p, void* workspace, int num_sms, cudaStream_t stream, int* launches);
size_t collapse_workspace_bytes(long long N, long long K);

// Appends the name of a kernel variant to this thread's record of what the current fc_run enqueues (fc_last_plan).
void note_kernel(const char* name);

// Stack of `mats` 16-bit matrices [C][P] -> [P][C] (layout.cu): the channels-last rewrite for CONV2D_NCHW.  C even.
// `beside_previous`: the kernel in front of this one in the stream shares no memory with it, so the two may overlap.
cudaError_t launch_cfirst_to_clast(const void* src, void* dst, long long mats, int C, int P, bool beside_previous, cudaStream_t stream,
                                   int* launches);

// Channels-last 16-bit image [batch][H][W][C] -> the same with a zero border of `pad` pixels (layout.cu).  C a multiple of 8.
cudaError_t launch_pad_image(const void* src, void* dst, long long batch, int H, int W, int C, int pad, int num_sms, cudaStream_t stream,
                             int* launches);

// Second pass of a wide GEMM + row softmax: per row, merges the tiles' (max, sum) pairs and rescales the stored
// exponentials of tile j by 2^((max_j - max_row) log2 e) / sum_row, in place.  `bn` = tile width in columns.
cudaError_t launch_softmax_rescale(void* out, int out_dt, const float2* stats, long long M, long long N, int tiles_n, int bn,
                                   int num_sms, cudaStream_t stream, int* launches);

// Zeroes `bytes` bytes (a multiple of 4, 4-byte aligned) with a kernel that lets the next kernel in the stream be
// scheduled at once: the pooled outputs of the convolution are cleared while its first tiles are in the main loop.
cudaError_t launch_zero_fill(void* ptr, size_t bytes, int num_sms, cudaStream_t stream, int* launches);

// tcgen05 GEMM family: plain epilogue (kMode 0), row softmax across tiles (1), conv + avg-pool (2)
struct TcParams {
    int mode;                   // 0 plain store, 1 row softmax, 2 conv + pooling, 3 row reduction to one value,
                                // 6 plain store with block-scaled E4M3 operands (scale tiles through a third and fourth tensor map),
                                // 7 plain store with 32-bit operands read as tf32 (K counts their elements)
    int M, N, K;                // GEMM view (conv: M = batch*OH*OW, N = Cout, K = R*S*Cin)
    int group_m;                // mode 0 raster: 256-row panels per sweep over the column tiles
    int in_dt;                  // FC_BF16 or FC_F16: storage of both MMA operands
    void* out; int out_dt;      // mode 0/1/3: [M,N] bf16 or f32 (mode 3: may be null).  mode 2: f32 [batch,Cout] (pre-zeroed)
    float* red;                 // mode 3: row reduction [M]
    int red_kind;               // mode 3: FC_RED_ROW_LOGSUMEXP, _SUM, _MAX or _MEAN
    DevOps ops;
    // mode 1
    float2* stats;              // (max, sum) per row and tile: [tiles_n][M] (tile-major, so that a warp reads and writes whole sectors), or [M][tiles_n][2] in the two-kernel softmax
    unsigned int* counters;     // [panels] arrivals; zero at launch, left at zero by a launch that completes
    unsigned int* departed;     // mode 1: [panels] tiles that have left the panel wait; same rule
    // mode 2
    int batch, H, W, Cin, Cout, R, S, stride, pad, OH, OW;
    float inv_hw;
    int pool;                   // mode 2: 0 global average pool; 2x2 max-pool (out pre-zeroed, values >= 0): 1 through atomics,
                                // 2 with the windows inside a tile finished on chip (narrow outputs)
    int m_rows;                 // mode 2: output positions that a CTA's tile stands for: 128, or with pool_whole the largest
                                // multiple of 2 * OW below (the tile still loads and multiplies 128 positions)
    int pool_whole;             // mode 2, pool == 2: tiles of whole row pairs (OH even): every window lies inside one tile, `out`
                                // needs no zeros, sees no atomics and may be a 16-bit tensor (out_dt)
    int two_pass;               // mode 1: rows wider than the tiles the SM pairs can hold at once: no waiting across tiles; every
                                // tile stores its exponentials against its own maximum and leaves (max, sum) in `stats`,
                                // launch_softmax_rescale finishes the rows
    int after_zero_fill;        // mode 2: launched programmatically behind the kernel that zeroes `out`; the epilogue warps wait
                                // for that kernel before their first update of `out`, everything else starts at once
    int a_packed;               // mode 2: 1 = a k-block of A is eight 8-channel chunks, one per filter tap (Cin == 8)
    int a_rowtaps;              // mode 2: 1 = a k-block is one filter row, or a 64-element piece of one: the S taps x Cin
                                // channels of a row are S * Cin contiguous elements in channels-last storage, fetched as
                                // (a piece of) one "pixel" of a tensor map whose pixels overlap (see row_taps in fc_api.cu)
    int* status;                // device status word
    long long dbg_trim;         // debug build: bytes by which the checks believe the main output to be shorter (testing)
    int expect_extra;           // testing only: arrivals a wait expects beyond those that will come (mode 1: the panel
                                // wait; other modes: the wait of a split tile's merging slice)
    // Split tiles (filled by the launcher when the scratch below is given and a split pays): tiles from
    // split_from on are cut into `split` slices along K.
    int split, split_from, split_kb;   // split_kb: k-blocks of each parking slice; the merging slice takes the rest
    float4* split_ws;           // kTcSplitUnits slots of 2 x 128 x BN fp32, or null: never split
    unsigned int* split_counters;   // kTcSplitUnits arrival counters (two per split tile); zero at launch, left at zero
};
// Scratch for split tiles: at most this many slice units per launch.
constexpr int kTcSplitUnits = 80;
constexpr size_t kTcSplitCounterBytes = 1024;
constexpr size_t kTcSplitBytes = kTcSplitCounterBytes + (size_t) kTcSplitUnits * 2 * 128 * 256 * 4;
cudaError_t launch_gemm_tc(const TcParams& p, const CUtensorMap& tmA, const CUtensorMap& tmB,
                           int bn, int num_sms, cudaStream_t stream, int* launches);
// Mode 6: `tmSA` / `tmSB` map the scale tiles written by launch_scale_tiles (rows of 128 words: one row per 128-row
// tile of A and k-block; one or two rows per column tile of B and k-block).  Column tiles are mx_tile_width(N) wide.
cudaError_t launch_gemm_tc_mx(const TcParams& p, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmSA,
                              const CUtensorMap& tmSB, int num_sms, cudaStream_t stream, int* launches);
// E8M0 scales [rows][K/32] -> tiles of 512 bytes per (128 rows, 128 elements of K), in the order the tensor core's
// scale columns want them: byte (r % 32) * 16 + (r / 32) * 4 + j holds the scale of row r of the tile and the j-th
// block of 32 elements.  Rows are grouped into row tiles of `tile_rows` (128 for A; the GEMM's column-tile width for B,
// 240 or 128), each ceil(tile_rows / 128) consecutive 512-byte tiles per k-block; positions without a row get the
// scale 1.  K a multiple of 128.  `beside_previous` as above.
cudaError_t launch_scale_tiles(const void* scales, void* tiles, long long rows, long long K, int tile_rows, bool beside_previous,
                               cudaStream_t stream, int* launches);
size_t scale_tiles_bytes(long long rows, long long K, int tile_rows);
inline int mx_tile_width(long long N) { return N <= 128 ? 128 : 240; }   // column-tile width of the block-scaled GEMM
size_t gemm_tc_smem_bytes(int bn);

// Back-to-back linear layers kept on chip (mlp_tc.cu): layer l maps width[l-1] (K0 for l = 0) to width[l]
struct MlpParams {
    int M, K0, layers;          // 2..4 layers
    int width[4];               // every width <= 256 and a multiple of 8
    int in_dt;                  // FC_BF16 or FC_F16: storage of x, of every weight matrix and of the activations between layers
    void* out; int out_dt;      // [M, width[layers-1]]
    DevOps seg[4];              // ops applied to the accumulator of layer l (no ADD_TENSOR)
    int* status;
};
cudaError_t launch_mlp_tc(const MlpParams& p, const CUtensorMap& tmX, const CUtensorMap* tmW, int num_sms, cudaStream_t stream,
                          int* launches);

// What launch_gemm_tc would do with `p` on the current device (no launch).
struct TcPlan {
    int bn, tiles, pairs;       // tile width, 256 x bn output tiles, CTA pairs launched
    int split, split_tiles, split_kb;   // slices per split tile (1: none), tiles that are split, k-blocks per parking slice
    int num_kb;                 // k-blocks of a whole tile
};
cudaError_t plan_gemm_tc(const TcParams& p, int bn, int num_sms, TcPlan* plan);

}  // namespace fc
