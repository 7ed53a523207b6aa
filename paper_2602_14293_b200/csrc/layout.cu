// Channel-first -> channels-last rewrite of 16-bit tensors, the pre-pass of the CONV2D_NCHW producer.
//
// Both operands of the convolution are, per outer index, a [C][P] matrix that the tensor-core kernel wants as
// [P][C]: the image per batch entry (P = H*W pixels) and the weights per output channel (P = R*S taps).  One
// kernel transposes a stack of such matrices through a 64 x 64 shared-memory tile: reads are contiguous along P
// (four pixels per load where the rows allow it), writes are contiguous along C (two channels per 32-bit store,
// 128 bytes per warp; C is a multiple of 8 for the convolution).
// HBM-bound: every element is read once and written once.
#include "fc_internal.h"

#include <cstdint>

namespace fc {
namespace {

constexpr int kTile = 64;
constexpr int kPitch = kTile + 2;   // 33 words per row: the column reads of the store phase touch each bank at most twice

// kVec = 4: rows of P elements start on 8-byte boundaries (P % 4 == 0), four pixels per load; kVec = 1: any P;
// kVec = 0: P <= 64 (filter taps), where the 64 rows of a tile are one contiguous run of 64 P elements that is
// copied linearly (pitch P in shared memory) instead of row by row with most lanes idle.
// All loads of a thread are issued before the first shared-memory store, so that a block keeps its whole
// tile in flight instead of paying the memory latency once per row.
template <int kVec>
__global__ void __launch_bounds__(256) cfirst_to_clast_kernel(const unsigned short* __restrict__ src, unsigned short* __restrict__ dst,
                                                              int C, int P, int tiles_p) {
    __shared__ __align__(16) unsigned short tile[kTile][kPitch];   // [c][p]
    const long long mat = blockIdx.x / tiles_p;
    const int p0 = (int) (blockIdx.x % tiles_p) * kTile, c0 = blockIdx.y * kTile;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned short* s = src + mat * (long long) C * P;
    unsigned short* d = dst + mat * (long long) C * P;
    if constexpr (kVec == 4) {
        const int pv = 4 * (threadIdx.x & 15), cr = threadIdx.x >> 4;
        uint2 v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = cr + 16 * i;
            v[i] = make_uint2(0u, 0u);
            if (c0 + c < C && p0 + pv < P) v[i] = *reinterpret_cast<const uint2*>(s + (long long) (c0 + c) * P + p0 + pv);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            unsigned int* w = reinterpret_cast<unsigned int*>(&tile[cr + 16 * i][pv]);
            w[0] = v[i].x;
            w[1] = v[i].y;
        }
    } else if constexpr (kVec == 0) {
        unsigned short* flat = &tile[0][0];
        const int n = min(kTile, C - c0) * P;
        const unsigned short* run = s + (long long) c0 * P;
        unsigned short v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int idx = threadIdx.x + 256 * i;
            v[i] = 0;
            if (idx < n) v[i] = run[idx];
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) flat[threadIdx.x + 256 * i] = v[i];
    } else {
        unsigned short v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int c = warp + 8 * (i >> 1), p = lane + 32 * (i & 1);
            v[i] = 0;
            if (c0 + c < C && p0 + p < P) v[i] = s[(long long) (c0 + c) * P + p0 + p];
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) tile[warp + 8 * (i >> 1)][lane + 32 * (i & 1)] = v[i];
    }
    __syncthreads();
    // Under a programmatic launch (see the launcher) this kernel ran beside the tail of the one in front, with
    // which it shares nothing; it must not be seen as complete before that one is.  A no-op otherwise.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int c = 2 * lane;   // C is even: a pair of channels is either inside or outside
    if constexpr (kVec == 0) {
        const unsigned short* flat = &tile[0][0];
        if (c0 + c < C)
            for (int p = warp; p < P; p += 8) {
                const unsigned int v = (unsigned int) flat[c * P + p] | ((unsigned int) flat[(c + 1) * P + p] << 16);
                *reinterpret_cast<unsigned int*>(d + (long long) p * C + c0 + c) = v;
            }
    } else if (c0 + c < C) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int p = warp + 8 * i;
            if (p0 + p < P) {
                const unsigned int v = (unsigned int) tile[c][p] | ((unsigned int) tile[c + 1][p] << 16);
                *reinterpret_cast<unsigned int*>(d + (long long) (p0 + p) * C + c0 + c) = v;
            }
        }
    }
}

__global__ void __launch_bounds__(256) zero_fill_kernel(uint32_t* ptr, size_t words) {
    // the kernel behind this one may be scheduled now; it waits (griddepcontrol.wait) where it first needs the zeros
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const size_t stride = (size_t) gridDim.x * blockDim.x;
    size_t i = (size_t) blockIdx.x * blockDim.x + threadIdx.x;
    if ((reinterpret_cast<uintptr_t>(ptr) & 15) == 0) {
        uint4* p4 = reinterpret_cast<uint4*>(ptr);
        const size_t quads = words >> 2;
        for (size_t q = i; q < quads; q += stride) p4[q] = make_uint4(0u, 0u, 0u, 0u);
        for (size_t w = (quads << 2) + i; w < words; w += stride) ptr[w] = 0u;
    } else {
        for (; i < words; i += stride) ptr[i] = 0u;
    }
}

// One thread per (position of a scale tile, four k-blocks): reads the 16 scale bytes of its row for those k-blocks and
// writes one word into each of their four tiles.  A tile of `tile_rows` rows (128 for A, the GEMM's column-tile width for
// B) is ceil(tile_rows / 128) consecutive 512-byte tiles; positions that stand for no row get the scale 1.
__global__ void __launch_bounds__(256) scale_tiles_kernel(const uint8_t* __restrict__ scales, uint32_t* __restrict__ tiles, long long rows,
                                                          int blocks32, int num_kb, int tile_rows, long long positions) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int groups = (num_kb + 3) >> 2;
    const int parts = (tile_rows + 127) >> 7;            // 512-byte tiles per row tile
    const long long idx = (long long) blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= positions * groups) return;
    const long long pos = idx / groups;                  // (row tile, part, row within the part)
    const int g = (int) (idx - pos * groups);
    const long long tile = pos / (parts * 128);
    const int within = (int) (pos - tile * (parts * 128)), part = within >> 7, rr = within & 127;
    const int in_tile = part * 128 + rr;
    const long long r = tile * tile_rows + in_tile;
    uint32_t w[4] = {0x7f7f7f7fu, 0x7f7f7f7fu, 0x7f7f7f7fu, 0x7f7f7f7fu};   // scale 1 where there is no row
    if (in_tile < tile_rows && r < rows) {
        const uint8_t* src = scales + r * blocks32 + 16 * g;
        if (16 * g + 16 <= blocks32 && (reinterpret_cast<uintptr_t>(src) & 15) == 0) {
            const uint4 q = *reinterpret_cast<const uint4*>(src);
            w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w;
        } else {
            for (int i = 0; i < 4; ++i)
                if (16 * g + 4 * i + 4 <= blocks32) w[i] = (uint32_t) src[4 * i] | (uint32_t) src[4 * i + 1] << 8 | (uint32_t) src[4 * i + 2] << 16 | (uint32_t) src[4 * i + 3] << 24;
        }
    }
    const int word = (rr & 31) * 4 + (rr >> 5);
    for (int i = 0; i < 4; ++i) {
        const int kb = 4 * g + i;
        if (kb < num_kb) tiles[((tile * num_kb + kb) * parts + part) * 128 + word] = w[i];
    }
}

// fp32 operands for the tensor cores.  A 32-bit value x is cut into hi (sign, exponent and the ten mantissa bits that
// kind::tf32 reads) and lo = x - hi (exact in fp32; its own upper bits are what the tensor core reads of it).  With
// A' = [A_lo | A_hi | A_hi] and B' = [B_hi | B_lo | B_hi] along K, A' B'^T = A_hi B_hi + A_hi B_lo + A_lo B_hi: the
// fp32 product up to the lo x lo terms and the bits of lo beyond its own ten (2^-21 relative per product), accumulated
// in fp32, the small terms first.  One thread per four consecutive k of a row; K is a multiple of 4.
__global__ void __launch_bounds__(256) split_tf32_kernel(const float* __restrict__ x, float* __restrict__ y, long long rows, int K, int is_b) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int quads = K >> 2;
    const long long idx = (long long) blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * quads) return;
    const long long r = idx / quads;
    const int q = (int) (idx - r * quads);
    const float4 v = __ldg(reinterpret_cast<const float4*>(x + r * K) + q);
    const float in[4] = {v.x, v.y, v.z, v.w};
    float hi[4], lo[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t b = __float_as_uint(in[j]);
        const bool finite = (b & 0x7f800000u) != 0x7f800000u;
        // An infinity or a NaN goes to lo whole and leaves hi zero: it then meets only the other operand's hi, as in
        // the fp32 product (in hi it would also meet the other operand's lo, which is 0 for every value that tf32
        // represents exactly: inf x 0 = NaN where fp32 gives inf).  Two non-finite values at the same k give NaN.
        hi[j] = finite ? __uint_as_float(b & 0xffffe000u) : 0.0f;
        lo[j] = finite ? __uint_as_float(__float_as_uint(in[j] - hi[j]) & 0xffffe000u) : ((b & 0x007fffffu) ? __uint_as_float(0x7fc00000u) : in[j]);
    }
    const float4 h4 = make_float4(hi[0], hi[1], hi[2], hi[3]), l4 = make_float4(lo[0], lo[1], lo[2], lo[3]);
    float4* out = reinterpret_cast<float4*>(y + r * 3 * K);
    out[q] = is_b ? h4 : l4;
    out[quads + q] = is_b ? l4 : h4;
    out[2 * quads + q] = h4;
}

}  // namespace

size_t scale_tiles_bytes(long long rows, long long K, int tile_rows) {
    return (size_t) ((rows + tile_rows - 1) / tile_rows) * (size_t) ((tile_rows + 127) / 128) * (size_t) (K / 128) * 512;
}

cudaError_t launch_scale_tiles(const void* scales, void* tiles, long long rows, long long K, int tile_rows, bool beside_previous,
                               cudaStream_t stream, int* launches) {
    const int num_kb = (int) (K / 128), groups = (num_kb + 3) / 4;
    const long long positions = (rows + tile_rows - 1) / tile_rows * ((tile_rows + 127) / 128) * 128, total = positions * groups;
    if (K % 128 || total > 0x7fffffffLL * 256) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned) ((total + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = beside_previous ? 1 : 0;
    note_kernel("scale_tiles");
    ++*launches;
    return cudaLaunchKernelEx(&cfg, scale_tiles_kernel, (const uint8_t*) scales, (uint32_t*) tiles, rows, (int) (K / 32), num_kb, tile_rows, positions);
}

cudaError_t launch_split_tf32(const float* x, float* y, long long rows, long long K, bool is_b, bool beside_previous, cudaStream_t stream,
                              int* launches) {
    const long long total = rows * (K / 4);
    if (K % 4 || K > 0x7fffffffLL / 3 || total > 0x7fffffffLL * 256) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned) ((total + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = beside_previous ? 1 : 0;
    note_kernel("split_tf32");
    ++*launches;
    return cudaLaunchKernelEx(&cfg, split_tf32_kernel, x, y, rows, (int) K, is_b ? 1 : 0);
}

// A channels-last image with its zero border written out: [batch][H + 2 pad][W + 2 pad][C], C a multiple of 8
// (16-byte copies).  See padded_rows in fc_api.cu.
__global__ void __launch_bounds__(256) pad_image_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, long long batch, int H, int W,
                                                        int c8, int pad) {
    const int Hp = H + 2 * pad, Wp = W + 2 * pad;
    const long long total = batch * Hp * Wp * c8;
    const long long stride = (long long) gridDim.x * blockDim.x;
    for (long long i = (long long) blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int c = (int) (i % c8);
        const long long px = i / c8;
        const int w = (int) (px % Wp) - pad;
        const long long t = px / Wp;
        const int h = (int) (t % Hp) - pad;
        const long long b = t / Hp;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (h >= 0 && h < H && w >= 0 && w < W) v = __ldg(src + ((b * H + h) * W + w) * c8 + c);
        dst[i] = v;
    }
}

cudaError_t launch_pad_image(const void* src, void* dst, long long batch, int H, int W, int C, int pad, int num_sms, cudaStream_t stream,
                             int* launches) {
    if ((C & 7) || (reinterpret_cast<uintptr_t>(src) & 15) || (reinterpret_cast<uintptr_t>(dst) & 15)) return cudaErrorInvalidValue;
    const long long total = batch * (H + 2 * pad) * (W + 2 * pad) * (C / 8);
    long long blocks = (total + 255) / 256;
    if (blocks < 1) blocks = 1;
    if (blocks > (long long) num_sms * 8) blocks = (long long) num_sms * 8;
    note_kernel("pad_image");
    pad_image_kernel<<<(unsigned) blocks, 256, 0, stream>>>((const uint4*) src, (uint4*) dst, batch, H, W, C / 8, pad);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_zero_fill(void* ptr, size_t bytes, int num_sms, cudaStream_t stream, int* launches) {
    const size_t words = bytes / 4;
    size_t blocks = (words / 4 + 255) / 256;
    if (blocks < 1) blocks = 1;
    if (blocks > (size_t) num_sms * 4) blocks = (size_t) num_sms * 4;
    note_kernel("zero_fill");
    zero_fill_kernel<<<(unsigned) blocks, 256, 0, stream>>>((uint32_t*) ptr, words);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_cfirst_to_clast(const void* src, void* dst, long long mats, int C, int P, bool beside_previous, cudaStream_t stream,
                                   int* launches) {
    const int tiles_p = (P + kTile - 1) / kTile;
    const long long gx = mats * tiles_p;
    if (gx > 0x7fffffffLL || (C & 1)) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned) gx, (unsigned) ((C + kTile - 1) / kTile));
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    // `beside_previous`: the kernel in front of this one in the stream touches none of this one's memory (the
    // other operand's transposition), so this one's CTAs may start while that one drains
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = beside_previous ? 1 : 0;
    const unsigned short* s16 = (const unsigned short*) src;
    unsigned short* d16 = (unsigned short*) dst;
    ++*launches;
    note_kernel("cfirst_to_clast");
    if (P <= kTile && P % 4 != 0) return cudaLaunchKernelEx(&cfg, cfirst_to_clast_kernel<0>, s16, d16, C, P, tiles_p);
    if (P % 4 == 0 && reinterpret_cast<uintptr_t>(src) % 8 == 0) return cudaLaunchKernelEx(&cfg, cfirst_to_clast_kernel<4>, s16, d16, C, P, tiles_p);
    return cudaLaunchKernelEx(&cfg, cfirst_to_clast_kernel<1>, s16, d16, C, P, tiles_p);
}

}  // namespace fc
