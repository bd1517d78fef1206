// Shared declarations of the MoQE routed quantized-linear library (sm_100a).
//
// Packed expert layout (private to the library; the canonical view is what
// moqe_expert_export returns).  N and K are padded to multiples of 128
// (Np, Kp); padded codes are 0 and padded scales are 0.
//
//   tile (nt, kb)   : 128 output channels x 128 input features, contiguous,
//                     tiles ordered [nt][kb], tile_stride bytes apart  ->  one bulk copy per tile
//   blob  nb (0..7) : 16 channels x 128 k inside the tile, contiguous
//   piece (row, q)  : 32 codes of one channel: k = 128*kb + 32*G + 8*q + t,
//                     G = 0..3 ("chunk": 8 consecutive k), t = 0..7
//                     row = 16*nb + 8*half + r
//   slot            : q*8 + (r ^ 2q) (32 slots per half).  The xor makes the 16-byte slots
//                     bank-conflict free for both readers: lanes (r, q) = (lane/4, lane%4) of an
//                     mma.sync fragment and lanes (q, r') = (lane/8, lane%8) of the UMMA dequant warps
//
//   W4  blob 1024 B : [half][slot] 16 B = 4 words, word G = chunk G; code t sits in
//                     nibble t/2 (t even) or 4 + t/2 (t odd), so that
//                     ((w >> 4i) & 0x000F000F) yields the pair (t=2i, t=2i+1).
//   W8  blob 2048 B : [half][u][slot] 16 B, u = 0,1: bytes = chunk 2u (8 B) then chunk 2u+1.
//   W3  blob  768 B : [slot] 16 B = {A,B,C of half 0, A of half 1} then (at +512)
//                     [slot] 8 B = {B,C of half 1}.  A piece is three words A,B,C; code
//                     i = 8*G + t is the low (t even) / high (t odd) half of pair p = i/2:
//                     p < 15: word p/5, bits 3*(p%5) + 16*(i&1) .. +2
//                     p = 15: bit b of the code is bit 15 + 16*(i&1) of word b.
//   W2  blob  512 B : [slot] 16 B = {word 0, word 1 of half 0, word 0, word 1 of half 1}: one 16-byte load brings
//                     a lane the pieces of channel rows r and r + 8.  A piece is two words; word j holds chunks 2j
//                     and 2j+1; code i = 8*G + t is the low (t even) / high (t odd) half of field 4*(G&1) + t/2,
//                     bits 2*field .. +1 of its halfword, so that ((w >> 2f) & 0x00030003) yields a pair.
//
// This piece/k assignment serves both GEMM kernels: a lane of an mma.sync
// m16n8k16 fragment owns 4 k of every MMA (chunk halves), and every unpacked
// word is one 16-byte chunk of 8 consecutive k of a K-major UMMA operand tile.
//
// Scales and zero-points travel WITH the tile they belong to, so that one bulk copy brings
// everything a k-block needs: a tile is [codes][meta], meta = for each of the tile's groups
// (group 32: 4, group 64: 2, group >= 128: 1 -- a group wider than 128 k is repeated in each
// tile it spans) 128 fp16 scales followed, for asymmetric experts, by 128 bf16 zero-points
// (the integer zero-point; symmetric experts use 2^(bits-1)).  Per-channel experts have no
// per-tile meta: their scales / zero-points are plain [Np] arrays.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/moqe.h"

static __host__ __device__ inline int moqe_blob_bytes(int bits) { return 16 * 128 * bits / 8; }
static __host__ __device__ inline int moqe_tile_bytes(int bits) { return 128 * 128 * bits / 8; }   // codes only
static __host__ __device__ inline int moqe_groups_per_tile(int group) { return group == 0 ? 0 : (group >= 128 ? 1 : 128 / group); }
static __host__ __device__ inline int moqe_meta_group_bytes(int has_zeros) { return has_zeros ? 512 : 256; }
static __host__ __device__ inline int moqe_tile_stride(int bits, int group, int has_zeros) {
    return moqe_tile_bytes(bits) + moqe_groups_per_tile(group) * moqe_meta_group_bytes(has_zeros);
}

// What a kernel needs to know about one expert's device buffers.
struct ExpertDev {
    const uint8_t* tiles;           // [nt][kb] tiles of tile_stride bytes: codes then per-tile scales / zero-points
    const __half* scales_pc;        // per-channel experts only: [Np]
    const __nv_bfloat16* zeros_pc;  // per-channel asymmetric experts only: [Np]
    int bits;
    int group;                      // 0 = per channel
    int has_zeros;                  // asymmetric
    int tile_stride;
};

// scale / zero-point of channel row (0..127 inside the tile) for sub-group j of a tile in shared or global memory
static __device__ inline const __half* moqe_tile_scales(const unsigned char* tile, int bits, int has_zeros, int j) {
    return reinterpret_cast<const __half*>(tile + moqe_tile_bytes(bits) + j * moqe_meta_group_bytes(has_zeros));
}
static __device__ inline const __nv_bfloat16* moqe_tile_zeros(const unsigned char* tile, int bits, int j) {
    return reinterpret_cast<const __nv_bfloat16*>(tile + moqe_tile_bytes(bits) + j * 512 + 256);
}

struct moqe_expert {
    int N, K, bits, group, sym;   // as given by the caller (group 0 = per channel)
    int Np, Kp;                   // padded to multiples of 128
    int G;                        // real groups per row  (1 when group == 0)
    int device;
    uint8_t* tiles;               // packed tiles with their meta
    __half* scales_pc;            // per-channel: [Np], else nullptr
    __nv_bfloat16* zeros_pc;      // per-channel asymmetric: [Np], else nullptr
    size_t tiles_alloc, pc_alloc;
    ExpertDev dev() const {
        ExpertDev d;
        d.tiles = tiles; d.scales_pc = scales_pc; d.zeros_pc = zeros_pc; d.bits = bits; d.group = group;
        d.has_zeros = sym ? 0 : 1; d.tile_stride = moqe_tile_stride(bits, group, d.has_zeros);
        return d;
    }
};

namespace moqe {

// first device-detected error of this device (0 = none); kernels latch with atomicCAS
int* device_status_word();                 // allocates on first use for the current device
void count_launch(unsigned n = 1);

inline moqe_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? MOQE_OK : MOQE_ERR_CUDA; }

// route_permute.cu
moqe_status launch_sort(const int32_t* row_ids, int M, int E, int32_t* perm, int32_t* offsets, void* ws,
                        size_t ws_bytes, void* zero_region, size_t zero_bytes, void* Y_zero_invalid, int N,
                        cudaStream_t st);
size_t sort_workspace_bytes(int M, int E);
moqe_status launch_gather(const void* X, const int32_t* perm, const int32_t* offsets_E, int M, int C, void* Xp,
                          cudaStream_t st);

// 64-row boxes of the expert-sorted activations: copied to Xp only where the rows are not already consecutive in X
size_t gather_boxes_bytes(int M, int E);
moqe_status launch_gather_boxes(const void* X, const int32_t* perm, const int32_t* offsets, int M, int C, int E, void* Xp,
                                int32_t* box_src, cudaStream_t st);

// qgemm_stream.cu
size_t stream_workspace_bytes(int M, int Np, int E);
moqe_status launch_qgemm_stream(const void* X, int M, int N, int K, const moqe_expert* const* ex, int E, void* Y,
                                const int32_t* perm, const int32_t* offsets, void* ws, size_t ws_bytes,
                                cudaStream_t st);
size_t stream_zero_bytes(int M, int Np);
void stream_set_tile_cost(int bits, int cost);   // relative cost of one packed tile in the work split (measurement knob)

// qgemm_decode.cu: decode shapes -- at most DECODE_MAX_ROWS rows, experts per-channel or with groups of >= 128 k;
// nl layers that share the routing go down as one launch (ex[l * E + e] = expert e of layer l)
constexpr int DECODE_MAX_ROWS = 32;
bool decode_supported_multi(int M, const moqe_expert* const* ex, int nl, int E);
size_t decode_workspace_bytes(int M);
size_t decode_zero_bytes(int M);
moqe_status launch_qgemm_decode_multi(const void* const* X, int M, int nl, const moqe_expert* const* ex, int E,
                                      void* const* Y, const int32_t* perm, const int32_t* offsets, void* ws,
                                      size_t ws_bytes, cudaStream_t st);
moqe_status launch_qgemm_decode_ext(const void* const* X, int M, int nl, const moqe_expert* const* ex,
                                    const moqe_expert* const* ex2, int E, void* const* Y, const void* const* R,
                                    const int32_t* perm, const int32_t* offsets, void* ws, size_t ws_bytes, cudaStream_t st);
void decode_set_tile_cost(int bits, int cost);   // relative cost of one super-tile in the work split, by code width

// quantize.cu: a plain bf16 copy Wd[Np][2 Kp] (hi | lo halves) of a (small) expert and its per-channel output scale, for qgemm_dense.cu
moqe_status launch_dense_unpack(const moqe_expert* const* ex, int E, uint16_t* Wd, float* col_scale, cudaStream_t st);   // experts that agree on N and K, one launch: Wd[E][Np][2 Kp], col_scale[E][Np]

// qgemm_dense.cu: large batches on layers whose weights are small (activation-bound, e.g. 1x1 convolutions)
bool dense_supported(int M, int N, int K, const moqe_expert* const* ex, int E);
size_t dense_workspace_bytes(int M, int K, int E, int Np, int Kp);
moqe_status launch_qgemm_dense(const void* X, int M, int N, int K, const moqe_expert* const* ex, int E, void* Y,
                               const int32_t* perm, const int32_t* offsets, void* ws, size_t ws_bytes, cudaStream_t st);

// qgemm_tcgen05.cu
void tc_set_tile_tokens(int tn);   // 0 = automatic, else 128 or 256 (testing / measurement)
size_t tc_workspace_bytes(int M, int K, int E, int Np);
moqe_status launch_qgemm_tc(const void* X, int M, int N, int K, const moqe_expert* const* ex, int E, void* Y,
                            const int32_t* perm, const int32_t* offsets, void* ws, size_t ws_bytes,
                            cudaStream_t st);

__device__ __forceinline__ void latch_status(int* status, int code) {
    if (status) atomicCAS(status, 0, code);
}

}  // namespace moqe
