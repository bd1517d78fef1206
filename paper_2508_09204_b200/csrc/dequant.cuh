// Register-level unpacking of packed expert codes to exact bf16 integers (c - z).
//
// A "piece" is the 32 codes of one output channel that one lane owns inside a
// 16-channel x 128-k blob (see common.cuh): four chunks G = 0..3 of 8
// consecutive k.  unpack_chunk turns chunk G into four bf16x2 registers
// (k offsets {0,1},{2,3},{4,5},{6,7}) whose values are the exact integers
// c - z; the group scale is applied later in fp32, so the tensor cores only
// see exactly representable operands.
#pragma once
#include "common.cuh"

namespace moqe {

template <int BITS> struct PieceWords;
template <> struct PieceWords<4> { static constexpr int n = 4; };
template <> struct PieceWords<8> { static constexpr int n = 8; };
template <> struct PieceWords<3> { static constexpr int n = 3; };
template <> struct PieceWords<2> { static constexpr int n = 2; };

__device__ __forceinline__ uint32_t hsub2_bf16(uint32_t a, uint32_t b) {
    __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&a), y = *reinterpret_cast<__nv_bfloat162*>(&b);
    __nv_bfloat162 r = __hsub2(x, y);
    return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 r = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&r);
}

// z: the integer zero-point of this channel and group, as a float.
template <int BITS, int G>
__device__ __forceinline__ void unpack_chunk(const uint32_t (&w)[PieceWords<BITS>::n], float z, uint32_t (&out)[4]) {
    if constexpr (BITS == 4) {
        // 0x4300 | c is the bf16 number 128 + c; subtracting 128 + z (<= 143, exact in bf16) is exact.
        const uint32_t zz = pack_bf16x2(128.f + z, 128.f + z);
        const uint32_t v = w[G];
#pragma unroll
        for (int i = 0; i < 4; ++i) out[i] = hsub2_bf16(((v >> (4 * i)) & 0x000F000Fu) | 0x43004300u, zz);
    } else if constexpr (BITS == 2) {
        // word G / 2 holds chunks G & ~1 and G | 1: pair i of chunk G is field 4 * (G & 1) + i of both halfwords
        const uint32_t zz = pack_bf16x2(128.f + z, 128.f + z);
        const uint32_t v = w[G >> 1] >> (8 * (G & 1));
#pragma unroll
        for (int i = 0; i < 4; ++i) out[i] = hsub2_bf16(((v >> (2 * i)) & 0x00030003u) | 0x43004300u, zz);
    } else if constexpr (BITS == 3) {
        const uint32_t zz = pack_bf16x2(128.f + z, 128.f + z);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int p = 4 * G + i;                 // pair index inside the piece
            uint32_t v;
            if (p < 15) v = (w[p / 5] >> (3 * (p % 5))) & 0x00070007u;
            else v = ((w[0] >> 15) & 0x00010001u) | ((w[1] >> 14) & 0x00020002u) | ((w[2] >> 13) & 0x00040004u);
            out[i] = hsub2_bf16(v | 0x43004300u, zz);
        }
    } else {
        // A byte c zero-extended to 16 bits IS the bf16 number c * 2^-133 (subnormal below 128, and the encoding
        // runs on continuously into the first normal binade).  One fused multiply-add per PAIR of codes,
        // c * 2^-133 * 2^120 - z * 2^-13, gives (c - z) * 2^-13 exactly (|c - z| <= 255 has 8 significant bits);
        // the callers fold the factor 2^13 (W8_PRESCALE) into the fp32 scale.
        const float zs = z * 0.0001220703125f;                       // z * 2^-13, exact
        const uint32_t negz = pack_bf16x2(-zs, -zs);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t pair = __byte_perm(w[2 * G + (i >> 1)], 0u, (i & 1) ? 0x4342u : 0x4140u);   // {c_hi, c_lo} as 16-bit
            __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(&pair);
            const uint32_t k120 = 0x7B807B80u;                      // 2^120 in both halves
            __nv_bfloat162 r = __hfma2(v, *reinterpret_cast<const __nv_bfloat162*>(&k120),
                                       *reinterpret_cast<const __nv_bfloat162*>(&negz));
            out[i] = *reinterpret_cast<uint32_t*>(&r);
        }
    }
}

// what an 8-bit chunk unpacked by unpack_chunk must still be multiplied by
constexpr float W8_PRESCALE = 8192.f;

// Chunk G of a 4- or 3-bit piece as the bf16 numbers 128 + c (no zero-point): two instructions per pair.
// The caller removes (128 + z) * sum_k X with the help of a second MMA against an all-ones operand.
template <int BITS, int G>
__device__ __forceinline__ void unpack_chunk_biased(const uint32_t (&w)[PieceWords<BITS>::n], uint32_t (&out)[4]) {
    static_assert(BITS == 4 || BITS == 3 || BITS == 2, "biased form exists for 4-, 3- and 2-bit codes");
    if constexpr (BITS == 4) {
        const uint32_t v = w[G];
#pragma unroll
        for (int i = 0; i < 4; ++i) out[i] = ((v >> (4 * i)) & 0x000F000Fu) | 0x43004300u;
    } else if constexpr (BITS == 2) {
        const uint32_t v = w[G >> 1] >> (8 * (G & 1));
#pragma unroll
        for (int i = 0; i < 4; ++i) out[i] = ((v >> (2 * i)) & 0x00030003u) | 0x43004300u;
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int p = 4 * G + i;
            uint32_t v;
            if (p < 15) v = (w[p / 5] >> (3 * (p % 5))) & 0x00070007u;
            else v = ((w[0] >> 15) & 0x00010001u) | ((w[1] >> 14) & 0x00020002u) | ((w[2] >> 13) & 0x00040004u);
            out[i] = v | 0x43004300u;
        }
    }
}

// The packed words of one piece -- the 32 codes of channel row (half, r) and k quarter q of a 16-channel blob in
// shared memory -- at slot = q*8 + (r ^ 2q).
template <int BITS>
__device__ __forceinline__ void load_piece_smem(const unsigned char* blob, int half, int slot, uint32_t (&w)[PieceWords<BITS>::n]) {
    if constexpr (BITS == 4) {
        uint4 v = *reinterpret_cast<const uint4*>(blob + half * 512 + slot * 16);
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
    } else if constexpr (BITS == 8) {
        uint4 v = *reinterpret_cast<const uint4*>(blob + half * 1024 + slot * 16);
        uint4 u = *reinterpret_cast<const uint4*>(blob + half * 1024 + 512 + slot * 16);
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w; w[4] = u.x; w[5] = u.y; w[6] = u.z; w[7] = u.w;
    } else if constexpr (BITS == 2) {
        uint2 v = *reinterpret_cast<const uint2*>(blob + slot * 16 + half * 8);
        w[0] = v.x; w[1] = v.y;
    } else {
        if (half == 0) {
            uint4 v = *reinterpret_cast<const uint4*>(blob + slot * 16);
            w[0] = v.x; w[1] = v.y; w[2] = v.z;
        } else {
            w[0] = *reinterpret_cast<const uint32_t*>(blob + slot * 16 + 12);
            uint2 u = *reinterpret_cast<const uint2*>(blob + 512 + slot * 8);
            w[1] = u.x; w[2] = u.y;
        }
    }
}

// group index of chunk G of k-block kb:  per channel -> 0;  g = 32 -> 4*kb + G;  g = 64 -> 2*kb + G/2;
// g >= 128 -> 128*kb / g
__device__ __forceinline__ int group_of_chunk(int group, int kb, int G) {
    if (group == 0) return 0;
    if (group >= 128) return kb * 128 / group;
    return (kb * 128 + 32 * G) / group;
}

}  // namespace moqe
