// Expert construction: RTN quantizer, packer, canonical import / export.
//
// Section 3.1 of the paper: the experts are quantized variants of one
// full-precision model, built once and frozen.  The quantizer is affine
// round-to-nearest per (output channel, group of input features); see moqe.h
// for the exact arithmetic.  Every fp32 operation below is a single IEEE
// operation (explicit __f*_rn intrinsics, no fused multiply-add, no fast
// math), so codes, scales and zero-points are reproducible bit for bit.
#include <cstdio>
#include <cstring>
#include <new>

#include "dequant.cuh"

namespace moqe {
namespace {

// ---------------------------------------------------------------------------
// piece <-> packed words
// ---------------------------------------------------------------------------
// code index i = 8*G + t  (chunk G, position t)  <->  k = 128*kb + 32*G + 8*q + t
template <int BITS>
__device__ __forceinline__ void encode_piece(const uint32_t (&c)[32], uint32_t (&w)[PieceWords<BITS>::n]) {
    if constexpr (BITS == 4) {
#pragma unroll
        for (int G = 0; G < 4; ++G) {
            uint32_t v = 0;
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                int nib = (t & 1) ? 4 + (t >> 1) : (t >> 1);
                v |= (c[8 * G + t] & 0xFu) << (4 * nib);
            }
            w[G] = v;
        }
    } else if constexpr (BITS == 2) {
        w[0] = w[1] = 0;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int G = i >> 3, t = i & 7;
            w[G >> 1] |= (c[i] & 3u) << (2 * (4 * (G & 1) + (t >> 1)) + 16 * (t & 1));
        }
    } else if constexpr (BITS == 8) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            w[j] = (c[4 * j] & 0xFFu) | ((c[4 * j + 1] & 0xFFu) << 8) | ((c[4 * j + 2] & 0xFFu) << 16) |
                   ((c[4 * j + 3] & 0xFFu) << 24);
    } else {
        w[0] = w[1] = w[2] = 0;
#pragma unroll
        for (int i = 0; i < 30; ++i) {
            int p = i >> 1;
            w[p / 5] |= (c[i] & 7u) << (3 * (p % 5) + 16 * (i & 1));
        }
#pragma unroll
        for (int b = 0; b < 3; ++b) {
            w[b] |= ((c[30] >> b) & 1u) << 15;
            w[b] |= ((c[31] >> b) & 1u) << 31;
        }
    }
}

template <int BITS>
__device__ __forceinline__ void decode_piece(const uint32_t (&w)[PieceWords<BITS>::n], uint32_t (&c)[32]) {
    if constexpr (BITS == 4) {
#pragma unroll
        for (int G = 0; G < 4; ++G)
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                int nib = (t & 1) ? 4 + (t >> 1) : (t >> 1);
                c[8 * G + t] = (w[G] >> (4 * nib)) & 0xFu;
            }
    } else if constexpr (BITS == 2) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int G = i >> 3, t = i & 7;
            c[i] = (w[G >> 1] >> (2 * (4 * (G & 1) + (t >> 1)) + 16 * (t & 1))) & 3u;
        }
    } else if constexpr (BITS == 8) {
#pragma unroll
        for (int i = 0; i < 32; ++i) c[i] = (w[i >> 2] >> (8 * (i & 3))) & 0xFFu;
    } else {
#pragma unroll
        for (int i = 0; i < 30; ++i) {
            int p = i >> 1;
            c[i] = (w[p / 5] >> (3 * (p % 5) + 16 * (i & 1))) & 7u;
        }
        c[30] = c[31] = 0;
#pragma unroll
        for (int b = 0; b < 3; ++b) {
            c[30] |= ((w[b] >> 15) & 1u) << b;
            c[31] |= ((w[b] >> 31) & 1u) << b;
        }
    }
}

// address of the words of piece (half, slot) inside a blob
template <int BITS>
__device__ __forceinline__ void store_piece(uint8_t* blob, int half, int slot, const uint32_t (&w)[PieceWords<BITS>::n]) {
    if constexpr (BITS == 4) {
        *reinterpret_cast<uint4*>(blob + half * 512 + slot * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    } else if constexpr (BITS == 2) {
        *reinterpret_cast<uint2*>(blob + slot * 16 + half * 8) = make_uint2(w[0], w[1]);
    } else if constexpr (BITS == 8) {
        *reinterpret_cast<uint4*>(blob + half * 1024 + slot * 16) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(blob + half * 1024 + 512 + slot * 16) = make_uint4(w[4], w[5], w[6], w[7]);
    } else {
        uint32_t* a = reinterpret_cast<uint32_t*>(blob + slot * 16);
        uint32_t* b = reinterpret_cast<uint32_t*>(blob + 512 + slot * 8);
        if (half == 0) { a[0] = w[0]; a[1] = w[1]; a[2] = w[2]; }
        else           { a[3] = w[0]; b[0] = w[1]; b[1] = w[2]; }
    }
}

template <int BITS>
__device__ __forceinline__ void load_piece(const uint8_t* blob, int half, int slot, uint32_t (&w)[PieceWords<BITS>::n]) {
    if constexpr (BITS == 4) {
        uint4 v = *reinterpret_cast<const uint4*>(blob + half * 512 + slot * 16);
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
    } else if constexpr (BITS == 2) {
        uint2 v = *reinterpret_cast<const uint2*>(blob + slot * 16 + half * 8);
        w[0] = v.x; w[1] = v.y;
    } else if constexpr (BITS == 8) {
        uint4 v = *reinterpret_cast<const uint4*>(blob + half * 1024 + slot * 16);
        uint4 u = *reinterpret_cast<const uint4*>(blob + half * 1024 + 512 + slot * 16);
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w; w[4] = u.x; w[5] = u.y; w[6] = u.z; w[7] = u.w;
    } else {
        const uint32_t* a = reinterpret_cast<const uint32_t*>(blob + slot * 16);
        const uint32_t* b = reinterpret_cast<const uint32_t*>(blob + 512 + slot * 8);
        if (half == 0) { w[0] = a[0]; w[1] = a[1]; w[2] = a[2]; }
        else           { w[0] = a[3]; w[1] = b[0]; w[2] = b[1]; }
    }
}

// piece id -> coordinates.  Pieces are numbered so that consecutive threads own
// consecutive slots of one half of one blob (coalesced packed accesses).
struct PieceCoord { int nt, kb, nb, half, slot, q, r, n; size_t tile_index; };
__device__ __forceinline__ PieceCoord piece_coord(long long pid, int KB) {
    PieceCoord pc;
    pc.slot = (int)(pid & 31);
    pc.half = (int)((pid >> 5) & 1);
    pc.nb = (int)((pid >> 6) & 7);
    long long tile = pid >> 9;
    pc.kb = (int)(tile % KB);
    pc.nt = (int)(tile / KB);
    pc.q = pc.slot >> 3;
    pc.r = (pc.slot & 7) ^ (2 * pc.q);
    pc.n = pc.nt * 128 + pc.nb * 16 + pc.half * 8 + pc.r;
    pc.tile_index = (size_t)tile;
    return pc;
}

// ---------------------------------------------------------------------------
// K1a: per (channel, group) scale and zero-point.  One warp per group.
// ---------------------------------------------------------------------------
// where the scale / zero-point of (channel n, canonical group gi) live; a group wider than 128 k is
// stored once per tile it spans: copy 0 .. copies-1
struct MetaSlot { __half* s; __nv_bfloat16* z; };
__device__ __forceinline__ int meta_copies(int group) { return group > 128 ? group / 128 : 1; }
__device__ __forceinline__ MetaSlot meta_slot(uint8_t* tiles, __half* scales_pc, __nv_bfloat16* zeros_pc, int bits, int group,
                                              int has_zeros, int KB, int n, int gi, int copy) {
    MetaSlot m;
    if (group == 0) {
        m.s = scales_pc + n;
        m.z = has_zeros ? zeros_pc + n : nullptr;
        return m;
    }
    const int per_tile = moqe_groups_per_tile(group);
    const int kb = group >= 128 ? gi * (group / 128) + copy : gi / per_tile;
    const int j = group >= 128 ? 0 : gi % per_tile;
    uint8_t* tile = tiles + ((size_t)(n >> 7) * KB + kb) * (size_t)moqe_tile_stride(bits, group, has_zeros);
    uint8_t* meta = tile + moqe_tile_bytes(bits) + j * moqe_meta_group_bytes(has_zeros);
    m.s = reinterpret_cast<__half*>(meta) + (n & 127);
    m.z = has_zeros ? reinterpret_cast<__nv_bfloat16*>(meta + 256) + (n & 127) : nullptr;
    return m;
}

__global__ void rtn_scales_kernel(const float* __restrict__ W, int N, int K, int bits, int group, int G, int sym, int KB,
                                  uint8_t* __restrict__ tiles, __half* __restrict__ scales_pc,
                                  __nv_bfloat16* __restrict__ zeros_pc) {
    long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (warp >= (long long)N * G) return;
    int n = (int)(warp / G), gi = (int)(warp % G);
    const int g = group ? group : K;
    const float* w = W + (size_t)n * K + (size_t)gi * g;
    float lo = 0.f, hi = 0.f, a = 0.f;
    for (int k = lane; k < g; k += 32) {
        float v = w[k];
        lo = fminf(lo, v);
        hi = fmaxf(hi, v);
        a = fmaxf(a, fabsf(v));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
    }
    if (lane != 0) return;
    const int L = (1 << bits) - 1;
    const int qmax = (1 << (bits - 1)) - 1;
    float s32 = sym ? __fdiv_rn(a, (float)qmax) : __fdiv_rn(__fsub_rn(hi, lo), (float)L);
    __half sh = __float2half_rn(s32);
    float s = __half2float(sh);
    if (!(s > 0.f) || isinf(s)) { sh = __float2half_rn(1.0f); s = 1.0f; }
    int z = 0;
    if (!sym) {
        z = (int)rintf(__fdiv_rn(-lo, s));
        z = max(0, min(L, z));
    }
    for (int c = 0; c < meta_copies(group); ++c) {
        MetaSlot m = meta_slot(tiles, scales_pc, zeros_pc, bits, group, !sym, KB, n, gi, c);
        *m.s = sh;
        if (!sym) *m.z = __float2bfloat16_rn((float)z);            // exact: z <= 255
    }
}

// ---------------------------------------------------------------------------
// K1b: codes + packing (FROM_CODES: canonical codes are given, only pack)
// ---------------------------------------------------------------------------
template <int BITS, bool FROM_CODES>
__global__ void encode_pack_kernel(const float* __restrict__ W, const uint8_t* __restrict__ canon, int N, int K,
                                   int g /*0 = per channel*/, int sym, int KB, uint8_t* __restrict__ tiles,
                                   __half* __restrict__ scales_pc, __nv_bfloat16* __restrict__ zeros_pc, long long npieces) {
    long long pid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (pid >= npieces) return;
    PieceCoord pc = piece_coord(pid, KB);
    constexpr int L = (1 << BITS) - 1;
    constexpr int half_code = 1 << (BITS - 1);
    constexpr int qmax = half_code - 1;
    uint32_t c[32];
#pragma unroll
    for (int G = 0; G < 4; ++G) {
        int k0 = pc.kb * 128 + 32 * G + 8 * pc.q;
        bool live = (pc.n < N) && (k0 < K);            // K % 8 == 0: a chunk is wholly inside or outside
        if (!live) {
#pragma unroll
            for (int t = 0; t < 8; ++t) c[8 * G + t] = 0;
            continue;
        }
        if constexpr (FROM_CODES) {
            uint2 v = *reinterpret_cast<const uint2*>(canon + (size_t)pc.n * K + k0);
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                c[8 * G + t] = (v.x >> (8 * t)) & 0xFFu;
                c[8 * G + 4 + t] = (v.y >> (8 * t)) & 0xFFu;
            }
        } else {
            MetaSlot m = meta_slot(tiles, scales_pc, zeros_pc, BITS, g, !sym, KB, pc.n, g ? k0 / g : 0, 0);
            float s = __half2float(*m.s);
            int z = sym ? half_code : (int)__bfloat162float(*m.z);
            const float4* src = reinterpret_cast<const float4*>(W + (size_t)pc.n * K + k0);
            float4 v0 = src[0], v1 = src[1];
            float wv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                int q = (int)rintf(__fdiv_rn(wv[t], s));
                if (sym) q = max(-qmax, min(qmax, q)) + half_code;
                else     q = max(0, min(L, q + z));
                c[8 * G + t] = (uint32_t)q;
            }
        }
    }
    uint32_t w[PieceWords<BITS>::n];
    encode_piece<BITS>(c, w);
    store_piece<BITS>(tiles + pc.tile_index * (size_t)moqe_tile_stride(BITS, g, !sym) + pc.nb * moqe_blob_bytes(BITS), pc.half,
                      pc.slot, w);
}

template <int BITS>
__global__ void unpack_kernel(const uint8_t* __restrict__ tiles, int N, int K, int KB, int tile_stride,
                              uint8_t* __restrict__ canon, long long npieces) {
    long long pid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (pid >= npieces) return;
    PieceCoord pc = piece_coord(pid, KB);
    if (pc.n >= N) return;
    uint32_t w[PieceWords<BITS>::n];
    load_piece<BITS>(tiles + pc.tile_index * (size_t)tile_stride + pc.nb * moqe_blob_bytes(BITS), pc.half, pc.slot, w);
    uint32_t c[32];
    decode_piece<BITS>(w, c);
#pragma unroll
    for (int G = 0; G < 4; ++G) {
        int k0 = pc.kb * 128 + 32 * G + 8 * pc.q;
        if (k0 >= K) continue;
        uint2 v;
        v.x = c[8 * G] | (c[8 * G + 1] << 8) | (c[8 * G + 2] << 16) | (c[8 * G + 3] << 24);
        v.y = c[8 * G + 4] | (c[8 * G + 5] << 8) | (c[8 * G + 6] << 16) | (c[8 * G + 7] << 24);
        *reinterpret_cast<uint2*>(canon + (size_t)pc.n * K + k0) = v;
    }
}

// canonical [N][G] fp16 scales / zero-points  <->  the per-tile (or per-channel) device copies
__global__ void meta_export_kernel(const uint8_t* __restrict__ tiles, const __half* __restrict__ scales_pc,
                                   const __nv_bfloat16* __restrict__ zeros_pc, int N, int G, int KB, int bits, int group, int sym,
                                   uint16_t* __restrict__ scales_out, uint16_t* __restrict__ zeros_out) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)N * G) return;
    int n = (int)(i / G), gi = (int)(i % G);
    MetaSlot m = meta_slot(const_cast<uint8_t*>(tiles), const_cast<__half*>(scales_pc), const_cast<__nv_bfloat16*>(zeros_pc), bits,
                           group, !sym, KB, n, gi, 0);
    if (scales_out) scales_out[i] = __half_as_ushort(*m.s);
    if (zeros_out) {
        float z = sym ? (float)(1 << (bits - 1)) : __bfloat162float(*m.z);
        zeros_out[i] = __half_as_ushort(__float2half_rn(z));
    }
}

__global__ void meta_import_kernel(const uint16_t* __restrict__ scales_in, const uint16_t* __restrict__ zeros_in, int N, int G,
                                   int KB, int bits, int group, int sym, uint8_t* __restrict__ tiles,
                                   __half* __restrict__ scales_pc, __nv_bfloat16* __restrict__ zeros_pc) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)N * G) return;
    int n = (int)(i / G), gi = (int)(i % G);
    for (int c = 0; c < meta_copies(group); ++c) {
        MetaSlot m = meta_slot(tiles, scales_pc, zeros_pc, bits, group, !sym, KB, n, gi, c);
        *m.s = __ushort_as_half(scales_in[i]);
        if (!sym) *m.z = __float2bfloat16_rn(__half2float(__ushort_as_half(zeros_in[i])));
    }
}

moqe_status check_format(int N, int K, int bits, int group) {
    if (N <= 0 || K <= 0) return MOQE_ERR_SHAPE;
    if (bits != 2 && bits != 3 && bits != 4 && bits != 8) return MOQE_ERR_UNSUPPORTED;
    if (K % 8 != 0) return MOQE_ERR_UNSUPPORTED;
    if (group < 0) return MOQE_ERR_SHAPE;
    if (group != 0) {
        if (K % group != 0) return MOQE_ERR_SHAPE;
        if (!(group == 32 || group == 64 || group % 128 == 0)) return MOQE_ERR_UNSUPPORTED;
    }
    return MOQE_OK;
}

moqe_status alloc_expert(int N, int K, int bits, int group, int sym, cudaStream_t st, moqe_expert** out) {
    moqe_expert* e = new (std::nothrow) moqe_expert();
    if (!e) return MOQE_ERR_ALLOC;
    e->N = N; e->K = K; e->bits = bits; e->group = group; e->sym = sym ? 1 : 0;
    e->Np = (N + 127) / 128 * 128;
    e->Kp = (K + 127) / 128 * 128;
    e->G = group ? K / group : 1;
    e->tiles = nullptr; e->scales_pc = nullptr; e->zeros_pc = nullptr;
    if (cudaGetDevice(&e->device) != cudaSuccess) { delete e; return MOQE_ERR_CUDA; }
    e->tiles_alloc = (size_t)(e->Np / 128) * (e->Kp / 128) * moqe_tile_stride(bits, group, !e->sym);
    e->pc_alloc = group == 0 ? (size_t)e->Np * 2 : 0;
    bool ok = cudaMalloc(&e->tiles, e->tiles_alloc) == cudaSuccess;
    if (ok && group == 0) {
        ok = cudaMalloc(&e->scales_pc, e->pc_alloc) == cudaSuccess &&
             (e->sym || cudaMalloc(&e->zeros_pc, e->pc_alloc) == cudaSuccess);
    }
    if (!ok) {
        cudaGetLastError();
        cudaFree(e->tiles); cudaFree(e->scales_pc); cudaFree(e->zeros_pc);
        delete e;
        return MOQE_ERR_ALLOC;
    }
    // padded channels / padded k: codes 0, scale 0, zero-point 0
    cudaMemsetAsync(e->tiles, 0, e->tiles_alloc, st);
    if (e->scales_pc) cudaMemsetAsync(e->scales_pc, 0, e->pc_alloc, st);
    if (e->zeros_pc) cudaMemsetAsync(e->zeros_pc, 0, e->pc_alloc, st);
    *out = e;
    return MOQE_OK;
}

template <bool FROM_CODES>
moqe_status launch_encode(const moqe_expert* e, const float* W, const uint8_t* canon, cudaStream_t st) {
    int KB = e->Kp / 128;
    long long npieces = (long long)(e->Np / 128) * KB * 512;
    unsigned blocks = (unsigned)((npieces + 127) / 128);
#define MOQE_ENC(B)                                                                                                  \
    encode_pack_kernel<B, FROM_CODES><<<blocks, 128, 0, st>>>(W, canon, e->N, e->K, e->group, e->sym, KB, e->tiles,   \
                                                              e->scales_pc, e->zeros_pc, npieces)
    if (e->bits == 4) MOQE_ENC(4);
    else if (e->bits == 8) MOQE_ENC(8);
    else if (e->bits == 2) MOQE_ENC(2);
    else MOQE_ENC(3);
#undef MOQE_ENC
    count_launch();
    return cuda_ok(cudaGetLastError());
}

}  // namespace
}  // namespace moqe

using namespace moqe;

extern "C" moqe_status moqe_quantize_rtn(const float* W, int N, int K, int bits, int group, int sym, void* stream,
                                         moqe_expert** out) {
    if (!W || !out) return MOQE_ERR_NULL;
    moqe_status s = check_format(N, K, bits, group);
    if (s != MOQE_OK) return s;
    if (reinterpret_cast<uintptr_t>(W) % 16 != 0) return MOQE_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    moqe_expert* e = nullptr;
    s = alloc_expert(N, K, bits, group, sym, st, &e);
    if (s != MOQE_OK) return s;
    long long warps = (long long)N * e->G;
    unsigned blocks = (unsigned)((warps * 32 + 255) / 256);
    rtn_scales_kernel<<<blocks, 256, 0, st>>>(W, N, K, bits, group, e->G, e->sym, e->Kp / 128, e->tiles, e->scales_pc,
                                              e->zeros_pc);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) { moqe_expert_destroy(e); return MOQE_ERR_CUDA; }
    s = launch_encode<false>(e, W, nullptr, st);
    if (s != MOQE_OK) { moqe_expert_destroy(e); return s; }
    *out = e;
    return MOQE_OK;
}

extern "C" moqe_status moqe_expert_import(int N, int K, int bits, int group, int sym, const uint8_t* codes,
                                          const uint16_t* scales_f16, const uint16_t* zeros_f16, void* stream,
                                          moqe_expert** out) {
    if (!codes || !scales_f16 || !out) return MOQE_ERR_NULL;
    if (!sym && !zeros_f16) return MOQE_ERR_NULL;
    moqe_status s = check_format(N, K, bits, group);
    if (s != MOQE_OK) return s;
    if (reinterpret_cast<uintptr_t>(codes) % 8 != 0) return MOQE_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    moqe_expert* e = nullptr;
    s = alloc_expert(N, K, bits, group, sym, st, &e);
    if (s != MOQE_OK) return s;
    long long n = (long long)N * e->G;
    meta_import_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(scales_f16, zeros_f16, N, e->G, e->Kp / 128, bits, group,
                                                                    e->sym, e->tiles, e->scales_pc, e->zeros_pc);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) { moqe_expert_destroy(e); return MOQE_ERR_CUDA; }
    s = launch_encode<true>(e, nullptr, codes, st);
    if (s != MOQE_OK) { moqe_expert_destroy(e); return s; }
    *out = e;
    return MOQE_OK;
}

extern "C" moqe_status moqe_expert_export(const moqe_expert* e, uint8_t* codes, uint16_t* scales_f16,
                                          uint16_t* zeros_f16, void* stream) {
    if (!e) return MOQE_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (codes) {
        if (reinterpret_cast<uintptr_t>(codes) % 8 != 0) return MOQE_ERR_UNSUPPORTED;
        int KB = e->Kp / 128;
        long long npieces = (long long)(e->Np / 128) * KB * 512;
        unsigned blocks = (unsigned)((npieces + 127) / 128);
        const int stride = moqe_tile_stride(e->bits, e->group, !e->sym);
        if (e->bits == 4) unpack_kernel<4><<<blocks, 128, 0, st>>>(e->tiles, e->N, e->K, KB, stride, codes, npieces);
        else if (e->bits == 8) unpack_kernel<8><<<blocks, 128, 0, st>>>(e->tiles, e->N, e->K, KB, stride, codes, npieces);
        else if (e->bits == 2) unpack_kernel<2><<<blocks, 128, 0, st>>>(e->tiles, e->N, e->K, KB, stride, codes, npieces);
        else unpack_kernel<3><<<blocks, 128, 0, st>>>(e->tiles, e->N, e->K, KB, stride, codes, npieces);
        count_launch();
    }
    if (scales_f16 || zeros_f16) {
        long long n = (long long)e->N * e->G;
        meta_export_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(e->tiles, e->scales_pc, e->zeros_pc, e->N, e->G,
                                                                        e->Kp / 128, e->bits, e->group, e->sym, scales_f16,
                                                                        zeros_f16);
        count_launch();
    }
    return cuda_ok(cudaGetLastError());
}

extern "C" moqe_status moqe_expert_info(const moqe_expert* e, int* N, int* K, int* bits, int* group, int* sym,
                                        size_t* code_bytes, size_t* meta_bytes, size_t* alloc_bytes) {
    if (!e) return MOQE_ERR_NULL;
    if (N) *N = e->N;
    if (K) *K = e->K;
    if (bits) *bits = e->bits;
    if (group) *group = e->group;
    if (sym) *sym = e->sym;
    if (code_bytes) *code_bytes = (size_t)e->N * e->K * e->bits / 8;
    if (meta_bytes) *meta_bytes = (size_t)e->N * e->G * 2 * (e->sym ? 1 : 2);
    if (alloc_bytes) *alloc_bytes = e->tiles_alloc + e->pc_alloc * (e->sym ? 1 : 2);
    return MOQE_OK;
}

extern "C" moqe_status moqe_expert_destroy(moqe_expert* e) {
    if (!e) return MOQE_ERR_NULL;
    cudaError_t a = cudaFree(e->tiles), b = cudaFree(e->scales_pc), c = cudaFree(e->zeros_pc);
    delete e;
    return (a == cudaSuccess && b == cudaSuccess && c == cudaSuccess) ? MOQE_OK : MOQE_ERR_CUDA;
}

// ---------------------------------------------------------------------------- dense copy of a small expert
// For layers whose weights are a few hundred kilobytes (1x1 convolutions) the routed product is bound by the
// activations, and the weights are best handed to the tensor cores as a plain bf16 matrix Wd[Np][Kp] (row = output
// channel, K contiguous).  Per-channel experts: Wd = c - z, an exact small integer, and col_scale[n] = the channel's
// scale, applied to the fp32 sums.  Grouped experts: s * (c - z) (exact in fp32) is split into two bf16 numbers,
// hi = bf16(w) in columns [0, Kp) and lo = bf16(w - hi) in columns [Kp, 2 Kp), and col_scale[n] = 1: the caller
// multiplies the activations by both halves, which leaves a relative error of 2^-17 per weight.  Rows are 2 Kp wide.
namespace moqe {
namespace {
struct DenseSrc {
    const uint8_t* tiles[MOQE_MAX_EXPERTS];
    const __half* scales_pc[MOQE_MAX_EXPERTS];
    const __nv_bfloat16* zeros_pc[MOQE_MAX_EXPERTS];
    int bits[MOQE_MAX_EXPERTS], group[MOQE_MAX_EXPERTS], sym[MOQE_MAX_EXPERTS];
};

template <int BITS>
__device__ __forceinline__ void dense_unpack_piece(const uint8_t* __restrict__ tiles, const __half* __restrict__ scales_pc,
                                                   const __nv_bfloat16* __restrict__ zeros_pc, int N, int K, int Kp, int KB, int group,
                                                   int sym, uint16_t* __restrict__ Wd, float* __restrict__ col_scale, long long pid) {
    PieceCoord pc = piece_coord(pid, KB);
    const int stride = moqe_tile_stride(BITS, group, !sym);
    uint32_t w[PieceWords<BITS>::n];
    load_piece<BITS>(tiles + pc.tile_index * (size_t)stride + pc.nb * moqe_blob_bytes(BITS), pc.half, pc.slot, w);
    uint32_t c[32];
    decode_piece<BITS>(w, c);
    const bool live = pc.n < N;
    if (pc.kb == 0 && pc.q == 0) col_scale[pc.n] = !live ? 0.f : (group == 0 ? __half2float(scales_pc[pc.n]) : 1.f);
#pragma unroll
    for (int G = 0; G < 4; ++G) {
        const int k0 = pc.kb * 128 + 32 * G + 8 * pc.q;
        uint32_t o[4] = {0u, 0u, 0u, 0u}, o2[4] = {0u, 0u, 0u, 0u};
        if (live && k0 < K) {
            float s = 1.f, z = (float)(1 << (BITS - 1));
            if (group == 0) {
                if (!sym) z = __bfloat162float(zeros_pc[pc.n]);
            } else {
                MetaSlot m = meta_slot(const_cast<uint8_t*>(tiles), nullptr, nullptr, BITS, group, !sym, KB, pc.n, k0 / group, 0);
                s = __half2float(*m.s);
                if (!sym) z = __bfloat162float(*m.z);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float w0 = s * ((float)c[8 * G + 2 * i] - z), w1 = s * ((float)c[8 * G + 2 * i + 1] - z);
                __nv_bfloat162 v = __floats2bfloat162_rn(w0, w1);
                o[i] = *reinterpret_cast<uint32_t*>(&v);
                if (group != 0) {
                    __nv_bfloat162 r = __floats2bfloat162_rn(w0 - __low2float(v), w1 - __high2float(v));
                    o2[i] = *reinterpret_cast<uint32_t*>(&r);
                }
            }
        }
        *reinterpret_cast<uint4*>(Wd + (size_t)pc.n * 2 * Kp + k0) = make_uint4(o[0], o[1], o[2], o[3]);
        *reinterpret_cast<uint4*>(Wd + (size_t)pc.n * 2 * Kp + Kp + k0) = make_uint4(o2[0], o2[1], o2[2], o2[3]);
    }
}

// blockIdx.y = expert
__global__ void dense_unpack_kernel(const __grid_constant__ DenseSrc src, int N, int K, int Np, int Kp, int KB,
                                    uint16_t* __restrict__ Wd, float* __restrict__ col_scale, long long npieces) {
    const long long pid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (pid >= npieces) return;
    const int e = blockIdx.y;
    uint16_t* wd = Wd + (size_t)e * Np * 2 * Kp;
    float* cs = col_scale + (size_t)e * Np;
    if (src.bits[e] == 4) dense_unpack_piece<4>(src.tiles[e], src.scales_pc[e], src.zeros_pc[e], N, K, Kp, KB, src.group[e], src.sym[e], wd, cs, pid);
    else if (src.bits[e] == 8) dense_unpack_piece<8>(src.tiles[e], src.scales_pc[e], src.zeros_pc[e], N, K, Kp, KB, src.group[e], src.sym[e], wd, cs, pid);
    else if (src.bits[e] == 2) dense_unpack_piece<2>(src.tiles[e], src.scales_pc[e], src.zeros_pc[e], N, K, Kp, KB, src.group[e], src.sym[e], wd, cs, pid);
    else dense_unpack_piece<3>(src.tiles[e], src.scales_pc[e], src.zeros_pc[e], N, K, Kp, KB, src.group[e], src.sym[e], wd, cs, pid);
}
}  // namespace

moqe_status launch_dense_unpack(const moqe_expert* const* ex, int E, uint16_t* Wd, float* col_scale, cudaStream_t st) {
    DenseSrc src;
    for (int e = 0; e < E; ++e) {
        src.tiles[e] = ex[e]->tiles; src.scales_pc[e] = ex[e]->scales_pc; src.zeros_pc[e] = ex[e]->zeros_pc;
        src.bits[e] = ex[e]->bits; src.group[e] = ex[e]->group; src.sym[e] = ex[e]->sym;
    }
    const int KB = ex[0]->Kp / 128;
    const long long npieces = (long long)(ex[0]->Np / 128) * KB * 512;
    dense_unpack_kernel<<<dim3((unsigned)((npieces + 127) / 128), E), 128, 0, st>>>(src, ex[0]->N, ex[0]->K, ex[0]->Np, ex[0]->Kp, KB, Wd,
                                                                                  col_scale, npieces);
    count_launch();
    return cuda_ok(cudaGetLastError());
}
}  // namespace moqe

// ---------------------------------------------------------------------------- expert residency
// Section 4.4 of the paper and its appendix table "Router model and expert loading overhead": one expert is kept on
// the GPU, the others wait in CPU RAM (or on disk) and are loaded when the routing changes.  A packed expert is a
// plain byte image (its tiles, and for per-channel experts the scale / zero-point arrays), so moving it is pure
// copy-engine work: to a file, to pinned host memory, and back on a side stream while the current layer runs.
namespace moqe {
namespace {

struct ImageHeader {
    char magic[8];                 // "MOQEXP1\0"
    int32_t layout;                // version of the packed layout this library writes
    int32_t N, K, bits, group, sym;
    uint64_t tiles_bytes, pc_bytes;
};
constexpr int32_t PACKED_LAYOUT_VERSION = 1;

ImageHeader header_of(const moqe_expert* e) {
    ImageHeader h = {};
    memcpy(h.magic, "MOQEXP1", 8);
    h.layout = PACKED_LAYOUT_VERSION;
    h.N = e->N; h.K = e->K; h.bits = e->bits; h.group = e->group; h.sym = e->sym;
    h.tiles_bytes = e->tiles_alloc; h.pc_bytes = e->pc_alloc;
    return h;
}
// does the header describe an expert this library would lay out in exactly these sizes?
moqe_status header_ok(const ImageHeader& h) {
    if (memcmp(h.magic, "MOQEXP1", 8) != 0 || h.layout != PACKED_LAYOUT_VERSION) return MOQE_ERR_UNSUPPORTED;
    moqe_status s = check_format(h.N, h.K, h.bits, h.group);
    if (s != MOQE_OK) return s;
    const size_t Np = (size_t)(h.N + 127) / 128 * 128, Kp = (size_t)(h.K + 127) / 128 * 128;
    const size_t tiles = (Np / 128) * (Kp / 128) * moqe_tile_stride(h.bits, h.group, !h.sym);
    const size_t pc = h.group == 0 ? Np * 2 : 0;
    return (h.tiles_bytes == tiles && h.pc_bytes == pc && (h.sym == 0 || h.sym == 1)) ? MOQE_OK : MOQE_ERR_SHAPE;
}
size_t image_bytes(const ImageHeader& h) { return (size_t)h.tiles_bytes + (size_t)h.pc_bytes * (h.sym ? 1 : 2); }

}  // namespace
}  // namespace moqe

// A packed expert parked in pinned host memory: header + byte image.
struct moqe_expert_host {
    moqe::ImageHeader h;
    uint8_t* image;                // pinned: tiles, then scales_pc, then zeros_pc
};

extern "C" moqe_status moqe_expert_offload(const moqe_expert* e, void* stream, moqe_expert_host** out) {
    if (!e || !out) return MOQE_ERR_NULL;
    moqe_expert_host* hx = new (std::nothrow) moqe_expert_host();
    if (!hx) return MOQE_ERR_ALLOC;
    hx->h = header_of(e);
    hx->image = nullptr;
    if (cudaMallocHost(&hx->image, image_bytes(hx->h)) != cudaSuccess) { cudaGetLastError(); delete hx; return MOQE_ERR_ALLOC; }
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t err = cudaMemcpyAsync(hx->image, e->tiles, e->tiles_alloc, cudaMemcpyDeviceToHost, st);
    if (err == cudaSuccess && e->scales_pc) err = cudaMemcpyAsync(hx->image + e->tiles_alloc, e->scales_pc, e->pc_alloc, cudaMemcpyDeviceToHost, st);
    if (err == cudaSuccess && e->zeros_pc) err = cudaMemcpyAsync(hx->image + e->tiles_alloc + e->pc_alloc, e->zeros_pc, e->pc_alloc, cudaMemcpyDeviceToHost, st);
    if (err == cudaSuccess) err = cudaStreamSynchronize(st);       // the image is complete when the call returns
    if (err != cudaSuccess) { cudaFreeHost(hx->image); delete hx; return MOQE_ERR_CUDA; }
    *out = hx;
    return MOQE_OK;
}

extern "C" moqe_status moqe_expert_prefetch(const moqe_expert_host* hx, void* stream, moqe_expert** out) {
    if (!hx || !out) return MOQE_ERR_NULL;
    moqe_status s = header_ok(hx->h);
    if (s != MOQE_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    moqe_expert* e = nullptr;
    s = alloc_expert(hx->h.N, hx->h.K, hx->h.bits, hx->h.group, hx->h.sym, st, &e);
    if (s != MOQE_OK) return s;
    cudaError_t err = cudaMemcpyAsync(e->tiles, hx->image, e->tiles_alloc, cudaMemcpyHostToDevice, st);
    if (err == cudaSuccess && e->scales_pc) err = cudaMemcpyAsync(e->scales_pc, hx->image + e->tiles_alloc, e->pc_alloc, cudaMemcpyHostToDevice, st);
    if (err == cudaSuccess && e->zeros_pc) err = cudaMemcpyAsync(e->zeros_pc, hx->image + e->tiles_alloc + e->pc_alloc, e->pc_alloc, cudaMemcpyHostToDevice, st);
    if (err != cudaSuccess) { moqe_expert_destroy(e); return MOQE_ERR_CUDA; }
    *out = e;
    return MOQE_OK;
}

extern "C" moqe_status moqe_expert_host_info(const moqe_expert_host* hx, int* N, int* K, int* bits, int* group, int* sym,
                                             size_t* image_bytes_out) {
    if (!hx) return MOQE_ERR_NULL;
    if (N) *N = hx->h.N;
    if (K) *K = hx->h.K;
    if (bits) *bits = hx->h.bits;
    if (group) *group = hx->h.group;
    if (sym) *sym = hx->h.sym;
    if (image_bytes_out) *image_bytes_out = image_bytes(hx->h);
    return MOQE_OK;
}

extern "C" moqe_status moqe_expert_host_destroy(moqe_expert_host* hx) {
    if (!hx) return MOQE_ERR_NULL;
    cudaError_t a = cudaFreeHost(hx->image);
    delete hx;
    return a == cudaSuccess ? MOQE_OK : MOQE_ERR_CUDA;
}

extern "C" moqe_status moqe_expert_host_save(const moqe_expert_host* hx, const char* path) {
    if (!hx || !path) return MOQE_ERR_NULL;
    FILE* f = fopen(path, "wb");
    if (!f) return MOQE_ERR_IO;
    const size_t n = image_bytes(hx->h);
    const bool ok = fwrite(&hx->h, sizeof(hx->h), 1, f) == 1 && (n == 0 || fwrite(hx->image, 1, n, f) == n);
    const bool closed = fclose(f) == 0;
    return ok && closed ? MOQE_OK : MOQE_ERR_IO;
}

extern "C" moqe_status moqe_expert_host_load(const char* path, moqe_expert_host** out) {
    if (!path || !out) return MOQE_ERR_NULL;
    FILE* f = fopen(path, "rb");
    if (!f) return MOQE_ERR_IO;
    ImageHeader h;
    if (fread(&h, sizeof(h), 1, f) != 1) { fclose(f); return MOQE_ERR_IO; }
    moqe_status s = header_ok(h);
    if (s != MOQE_OK) { fclose(f); return s; }
    // the file must hold exactly the image the header promises
    const size_t n = image_bytes(h);
    if (fseek(f, 0, SEEK_END) != 0 || (size_t)ftell(f) != sizeof(h) + n || fseek(f, (long)sizeof(h), SEEK_SET) != 0) { fclose(f); return MOQE_ERR_IO; }
    moqe_expert_host* hx = new (std::nothrow) moqe_expert_host();
    if (!hx) { fclose(f); return MOQE_ERR_ALLOC; }
    hx->h = h;
    hx->image = nullptr;
    if (cudaMallocHost(&hx->image, n ? n : 1) != cudaSuccess) { cudaGetLastError(); delete hx; fclose(f); return MOQE_ERR_ALLOC; }
    const bool ok = fread(hx->image, 1, n, f) == n;
    fclose(f);
    if (!ok) { cudaFreeHost(hx->image); delete hx; return MOQE_ERR_IO; }
    *out = hx;
    return MOQE_OK;
}
