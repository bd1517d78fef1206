// Shared declarations of the MoQE routed quantized-linear library (sm_100a).
//
// Packed expert layout (private to the library; the canonical view is what
// moqe_expert_export returns).  N and K are padded to multiples of 128
// (Np, Kp); padded codes are 0 and padded scales are 0.
//
//   tile (nt, kb)   : 128 output channels x 128 input features, contiguous,
//                     tiles ordered [nt][kb]  ->  one bulk copy per tile
//   blob  nb (0..7) : 16 channels x 128 k inside the tile, contiguous
//   piece (row, q)  : 32 codes of one channel: k = 128*kb + 32*G + 8*q + t,
//                     G = 0..3 ("chunk": 8 consecutive k), t = 0..7
//                     row = 16*nb + 8*half + r
//   slot            : q*8 + r (32 slots per half)
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
//
// This piece/k assignment serves both GEMM kernels: a lane of an mma.sync
// m16n8k16 fragment owns 4 k of every MMA (chunk halves), and every unpacked
// word is one 16-byte chunk of 8 consecutive k of a K-major UMMA operand tile.
//
//   scales_t [Gp][Np] fp16, zeros_t [Gp][Np] bf16 (the integer zero-point;
//   absent for symmetric experts whose zero-point is 2^(bits-1)).
//   Gp = 1 for per-channel experts, else Kp / group.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/moqe.h"

struct moqe_expert {
    int N, K, bits, group, sym;   // as given by the caller (group 0 = per channel)
    int Np, Kp;                   // padded to multiples of 128
    int G;                        // real groups per row  (1 when group == 0)
    int Gp;                       // allocated groups per row
    int device;
    uint8_t* codes;               // packed tiles
    __half* scales_t;             // [Gp][Np]
    __nv_bfloat16* zeros_t;       // [Gp][Np], nullptr when symmetric
    size_t codes_alloc, meta_alloc;
};

// What a GEMM kernel needs to know about one expert.
struct ExpertDev {
    const uint8_t* codes;
    const __half* scales_t;
    const __nv_bfloat16* zeros_t;   // nullptr: symmetric
    int bits;
    int group;                      // 0 = per channel
};

static __host__ __device__ inline int moqe_blob_bytes(int bits) { return 16 * 128 * bits / 8; }
static __host__ __device__ inline int moqe_tile_bytes(int bits) { return 128 * 128 * bits / 8; }

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

// qgemm_stream.cu
size_t stream_workspace_bytes(int M, int Np, int E);
moqe_status launch_qgemm_stream(const void* X, int M, int N, int K, const moqe_expert* const* ex, int E, void* Y,
                                const int32_t* perm, const int32_t* offsets, void* ws, size_t ws_bytes,
                                cudaStream_t st);
size_t stream_zero_bytes(int M, int Np);

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
