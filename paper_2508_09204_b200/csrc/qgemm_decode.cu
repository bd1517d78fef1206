// Routed dequant-GEMM for decode shapes (a GEMV-like, HBM-bound path) (at most 32 token rows in the batch): every touched
// expert's packed weights are streamed from HBM exactly once.
//
//   producer (1 thread)   : one bulk copy per packed 128x128-code tile (codes + the tile's scales / zero-points,
//                           contiguous in HBM) into a shared-memory ring guarded by full/empty mbarriers.  A stage
//                           holds a "super-tile": the tiles (nt, nt + 1) of one k-block.  The copies carry an L2
//                           evict-first policy: weights pass through L2 once.
//   16 consumer warps     : warp w owns one 16-channel blob of the super-tile.  A lane reads the codes of channel
//                           rows g and g + 8, k quarter t (its share of an m16n8k16 A fragment) with conflict-free
//                           128-bit shared loads, unpacks them in registers and issues warp-level tensor-core MMAs
//                           (fp16 operands, fp32 accumulation) against the token fragments; it applies the group's
//                           scale in fp32 once per k-block and keeps the running sums of its piece in registers.
//   2 service warps       : stage the token rows one chunk of k-blocks ahead, double buffered: gathered through
//                           `perm` (the fused permutation), converted from bf16 to scaled fp16 in MMA fragment order,
//                           with their sums.  Chunk descriptors travel with the buffers, so the consumers follow the
//                           work split without walking it themselves.
//
//   Unpacking costs 5 integer instructions per 8 four-bit codes (1 per 2 eight-bit codes, 23 per 32 three-bit
//   codes, 10 per 16 two-bit codes): a masked code dropped into the mantissa of the fp16 number 1024 becomes 1024 + c, or 1024 + 16c
//   for a code that sits four bits higher -- no shift, no subtraction.  The tensor core multiplies by token
//   values that were pre-scaled by 1/16 at exactly those k, and what the constants 1024 and the zero-point
//   contribute is removed in fp32 with per-(token, k-block) sums of the token values:
//     Y[m][n] = sum_G s[n][G] * ( sum_{k in G} A[n][k] * B[m][k]  -  1024 * S1[m][G]  -  z[n][G] * S0[m][G] )
//   A = 1024 + c / sigma_k,  B = sigma_k * x,  S1 = sum sigma_k x,  S0 = sum x.  All products are exact
//   (11-bit x 8-bit significands).  bf16 token values beyond the fp16 range (|x| > 65504) are outside the
//   kernel's domain: they turn into infinities.
//
// Work split ("stream-K" over super-tiles): the super-tiles of every (layer, expert) pair whose expert received
// rows form one sequence [pair][channel-tile pair][k-block] with a per-format cost; CTA c of G owns the
// super-tiles whose start cost lies in [c*C/G, (c+1)*C/G) -- the split follows the routing, so an expert
// without rows costs nothing and a batch routed to one expert still uses every SM.  A warp that holds only
// part of a segment parks its fp32 partial sums and bumps its arrival counter for that segment; whoever
// arrives last adds the parked sums in CTA order (deterministic) and stores bf16 rows at their original
// positions (the fused un-permutation).  Nobody waits for another CTA, so the kernel cannot stall whatever
// else occupies the device.
//
// Every mbarrier wait is bounded; on expiry the CTA raises its abort flag, latches MOQE_ERR_TIMEOUT, and
// every role leaves its loop.
//
// The operation is Section 3.1 of the paper (the selected quantization expert runs the sample); the paper
// describes no kernel.
#include <type_traits>

#include "common.cuh"
#include "ptx.cuh"

namespace moqe {
namespace {

constexpr int GV_CONS = 16;                                    // consumer warps
constexpr int GV_SERV = 2;                                     // service warps
constexpr int GV_THREADS = (GV_CONS + GV_SERV + 1) * 32;       // + the producer's warp
constexpr int GV_MAX_STAGES = 12;
constexpr int GV_XCHG_BYTES = 8 * 8 * 32 * 4;                  // gated pairs: [8 blobs][8 values][32 lanes] floats
constexpr int GV_XBUF = 32 * 1024;                             // one chunk of staged token rows
constexpr int GV_CHUNK_KB = 16;                                // k-blocks per chunk for one token block (8 for two)
constexpr int GV_SBUF = GV_CHUNK_KB * 8 * 2 * 4;               // the chunk's sums: [k-block][token block][t][4] floats
// a parked partial sum: 256 channels x 8 * NTMAX tokens
__host__ __device__ constexpr int gv_slot_floats(int ntmax) { return GV_CONS * ntmax * 4 * 32; }
constexpr int GV_MAX_GRID = 256;
constexpr int GV_PREFETCH_TILES = 4;                           // super-tiles asked of L2 before the dependency wait

// FUSED: the variant with gated pairs and residual adds (it gives 8 KB of the ring to the exchange buffer)
template <bool FUSED>
struct GvSmem {
    static constexpr int ring_bytes = (FUSED ? 150 : 158) * 1024;
    static constexpr int ring_off = 0;
    static constexpr int x_off = ring_bytes;
    static constexpr int s_off = x_off + 2 * GV_XBUF;
    static constexpr int xchg_off = s_off + 2 * GV_SBUF;
    static constexpr int desc_off = xchg_off + (FUSED ? GV_XCHG_BYTES : 0);   // 2 chunk descriptors of 32 bytes
    static constexpr int bar_off = desc_off + 2 * 32;                     // wfull[12] wempty[12] xfull[2] xempty[2]
    static constexpr int off_off = bar_off + (2 * GV_MAX_STAGES + 4) * 8;
    static constexpr int perm_off = off_off + (MOQE_MAX_EXPERTS + 2) * 4;
    static constexpr int pair_off = perm_off + DECODE_MAX_ROWS * 4;       // {tb, te} per pair
    static constexpr int base_off = pair_off + MOQE_MAX_EXPERTS * 8;     // cost before each pair (long long)
    static constexpr int misc_off = base_off + MOQE_MAX_EXPERTS * 8;     // C (long long), G, stages, stage bytes, abort
    static constexpr int ps_off = misc_off + 32;                         // the pairs' scalars (a copy of GvParams::ps)
    static constexpr int total = ps_off + MOQE_MAX_EXPERTS * 48;
    static constexpr int dyn_bytes = total;
};
static_assert(GvSmem<false>::dyn_bytes <= 227 * 1024 && GvSmem<true>::dyn_bytes <= 227 * 1024, "shared memory budget");

// what the kernel needs to know about a (layer, expert) pair besides pointers; copied to shared memory on entry
struct PairS {
    int bits, group, has_zeros, stride;     // the expert's format; bytes of one packed tile
    int N, K, KB, NT1;                      // the layer's shape; k-blocks; 128-channel tiles
    int rexp;                               // the routing expert whose rows the pair takes
    int w;                                  // cost of one super-tile
    int gated;                              // a gated pair (see tiles2)
    int pad;
};
static_assert(sizeof(PairS) == 48, "PairS is copied word by word");

struct GvParams {
    ExpertDev ex[MOQE_MAX_EXPERTS];         // per (layer, expert) pair
    PairS ps[MOQE_MAX_EXPERTS];
    const uint16_t* X[MOQE_MAX_EXPERTS];    // the layer's input and output
    uint16_t* Y[MOQE_MAX_EXPERTS];
    // A gated pair (tiles2 != nullptr): the pair's second expert (same format and shape), whose product multiplies
    // silu of the first one's; the super-tile is then {tile nt of the first, tile nt of the second}.
    const uint8_t* tiles2[MOQE_MAX_EXPERTS];
    const __half* scales_pc2[MOQE_MAX_EXPERTS];
    const __nv_bfloat16* zeros_pc2[MOQE_MAX_EXPERTS];
    const uint16_t* Res[MOQE_MAX_EXPERTS];  // residual added to the product before the rounding, or nullptr
    const int32_t* perm;
    const int32_t* offsets;
    float* partials;                        // [CTA][2][gv_slot_floats(NTMAX)]
    uint32_t* counters;                     // [CTA][warp]: arrivals for the segment whose head that CTA holds; zero on entry, left zero
    int* status;
    int M, R, P;                            // rows of the batch, routing experts, pairs
    int small;                              // (total cost) x (grid) fits 31 bits: the work split runs in 32-bit arithmetic
};

// one chunk of work: k-blocks [kbc, kbc + nkb) of segment (pair v, channel-tile pair nt2), part of the piece [kb0, kb1)
struct ChunkDesc { int v, nt2, kbc, nkb, kb0, kb1, valid, pad; };

// a walk over the CTA's super-tiles in [pair][channel-tile pair][k-block] order, run by run (a run = the k-blocks of
// one piece: contiguous in HBM)
struct GvWalk {
    int v, st, te, kb, KB, nt2;
    __device__ __forceinline__ void start() { v = -1; st = te = kb = nt2 = 0; KB = 1; }
    // opens the next run; returns false at the end.  `changed`: the run belongs to another pair than the last one
    __device__ __forceinline__ bool next(const int* s_pair, const PairS* ps, int P, bool& changed) {
        changed = false;
        if (v >= 0) st += run();
        if (v < 0 || st >= te) {
            do { ++v; } while (v < P && s_pair[2 * v + 1] <= s_pair[2 * v]);
            if (v >= P) return false;
            st = s_pair[2 * v]; te = s_pair[2 * v + 1]; KB = ps[v].KB;
            nt2 = st / KB; kb = st - nt2 * KB;
            changed = true;
        } else {
            kb = 0; ++nt2;
        }
        return true;
    }
    __device__ __forceinline__ int run() const { return min(KB - kb, te - st); }
};

__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t addr) {
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Constants of the unpacking, held in registers the compiler cannot see through: (v & mask) | 0x64006400 is ONE
// three-input logic instruction when mask and constant are registers, two when they are immediates.
struct GvConst {
    uint32_t base, m4lo, m4hi, m3a, m3b, m3c, m3s0, m3s1, m3s2, m2a, m2b, m2c;
    // only the constants of one code width are set (and live) at a time
    template <int BITS>
    __device__ __forceinline__ void init() {
        asm volatile("mov.u32 %0, 0x64006400;" : "=r"(base));
        if constexpr (BITS == 4) {
            asm volatile("mov.u32 %0, 0x000F000F;" : "=r"(m4lo));
            asm volatile("mov.u32 %0, 0x00F000F0;" : "=r"(m4hi));
        } else if constexpr (BITS == 3) {
            asm volatile("mov.u32 %0, 0x00070007;" : "=r"(m3a));
            asm volatile("mov.u32 %0, 0x00380038;" : "=r"(m3b));
            asm volatile("mov.u32 %0, 0x01C001C0;" : "=r"(m3c));
            asm volatile("mov.u32 %0, 0x00400040;" : "=r"(m3s0));
            asm volatile("mov.u32 %0, 0x00800080;" : "=r"(m3s1));
            asm volatile("mov.u32 %0, 0x01000100;" : "=r"(m3s2));
        } else if constexpr (BITS == 2) {
            asm volatile("mov.u32 %0, 0x00030003;" : "=r"(m2a));
            asm volatile("mov.u32 %0, 0x000C000C;" : "=r"(m2b));
            asm volatile("mov.u32 %0, 0x00300030;" : "=r"(m2c));
        }
    }
};
// (v & mask) | c: the fp16 numbers 1024 + (field value) in both halves, for a field inside the mantissa
__device__ __forceinline__ uint32_t and_or(uint32_t v, uint32_t mask, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(v), "r"(mask), "r"(c));
    return d;
}

// pairs 0..3 of one 4-bit word (8 consecutive k): {1024 + c, 1024 + 16c, 1024 + c, 1024 + 16c}
__device__ __forceinline__ void unpack_w4(const GvConst& k, uint32_t v, uint32_t (&o)[4]) {
    o[0] = and_or(v, k.m4lo, k.base);
    o[1] = and_or(v, k.m4hi, k.base);
    const uint32_t u = v >> 8;
    o[2] = and_or(u, k.m4lo, k.base);
    o[3] = and_or(u, k.m4hi, k.base);
}
// the 8 pairs of one 2-bit word (two chunks; pair f is field f of both halfwords, at bits 2f): 1024 + {1, 4, 16} * c --
// fields 0..2 straight from the word, 3..5 after a shift by 6, 6..7 after a shift by 12
__device__ __forceinline__ void unpack_w2(const GvConst& k, uint32_t v, uint32_t (&o)[8]) {
    o[0] = and_or(v, k.m2a, k.base);
    o[1] = and_or(v, k.m2b, k.base);
    o[2] = and_or(v, k.m2c, k.base);
    const uint32_t u = v >> 6;
    o[3] = and_or(u, k.m2a, k.base);
    o[4] = and_or(u, k.m2b, k.base);
    o[5] = and_or(u, k.m2c, k.base);
    const uint32_t t = v >> 12;
    o[6] = and_or(t, k.m2a, k.base);
    o[7] = and_or(t, k.m2b, k.base);
}
// pairs 0..3 of an 8-bit chunk held in two words: 1024 + c
__device__ __forceinline__ void unpack_w8(uint32_t w0, uint32_t w1, uint32_t (&o)[4]) {
    o[0] = __byte_perm(w0, 0x64646464u, 0x4140u);
    o[1] = __byte_perm(w0, 0x64646464u, 0x4342u);
    o[2] = __byte_perm(w1, 0x64646464u, 0x4140u);
    o[3] = __byte_perm(w1, 0x64646464u, 0x4342u);
}
// the 16 pairs of a 3-bit piece (words A, B, C): pair p < 15 is field p % 5 of word p / 5 -> 1024 + {1, 8, 64, 1, 8} * c;
// pair 15 is spread over bit 15 / 31 of the three words -> 1024 + 64c
__device__ __forceinline__ void unpack_w3(const GvConst& k, uint32_t A, uint32_t B, uint32_t C, uint32_t (&o)[16]) {
    const uint32_t w[3] = {A, B, C};
    uint32_t s0 = 0;
#pragma unroll
    for (int i = 0; i < 3; ++i) {
        const uint32_t u = w[i] >> 9;
        if (i == 0) s0 = u;
        o[5 * i + 0] = and_or(w[i], k.m3a, k.base);
        o[5 * i + 1] = and_or(w[i], k.m3b, k.base);
        o[5 * i + 2] = and_or(w[i], k.m3c, k.base);
        o[5 * i + 3] = and_or(u, k.m3a, k.base);
        o[5 * i + 4] = and_or(u, k.m3b, k.base);
    }
    uint32_t r = and_or(s0, k.m3s0, k.base);            // bit 15 / 31 of A -> bit 6 / 22: 64 * (code bit 0)
    r = and_or(B >> 8, k.m3s1, r);                      // of B -> bit 7 / 23
    r = and_or(C >> 7, k.m3s2, r);                      // of C -> bit 8 / 24
    o[15] = r;
}
// log2 of 1 / sigma for pair p (0..15) of a piece: how far the code sits above the mantissa's unit
__device__ __forceinline__ int sigma_shift(int bits, int p) {
    if (bits == 8) return 0;
    if (bits == 4) return (p & 1) ? 4 : 0;
    if (bits == 2) return (p & 7) < 6 ? 2 * ((p & 7) % 3) : 2 * ((p & 7) - 6);
    return p == 15 ? 6 : 3 * ((p % 5) % 3);
}

template <int BITS, int NT, bool GROUPED, bool ASYM>
struct GvTag {
    static constexpr int bits = BITS, nt = NT;
    static constexpr bool grouped = GROUPED, asym = ASYM;
};

// The MMAs of one tile for one lane: `blob` is the shared-memory address of the warp's blob, `xb` that of the
// lane's token fragments of this k-block.
// The same for more than two token blocks: the token fragments are fetched where they are used (holding them all
// would take 16 registers per block).
template <int BITS, int NT>
__device__ __forceinline__ void tile_mma_wide(const GvConst& kc, uint32_t blob, int slot16, uint32_t xb, float (&acc)[NT][4]) {
    auto step = [&](int G, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3) {
        // one 32-k group of both channel rows against every token block: a* = row g pairs 0..3, c* = row g + 8
#pragma unroll
        for (int tb = 0; tb < NT; ++tb) {
            const uint4 b = lds128(xb + ((tb * 4 + G) << 9));
            mma_f16(acc[tb], a0, c0, a1, c1, b.x, b.y);
            mma_f16(acc[tb], a2, c2, a3, c3, b.z, b.w);
        }
    };
    if constexpr (BITS == 4) {
        const uint4 w0 = lds128(blob + slot16), w1 = lds128(blob + 512 + slot16);
        const uint32_t a0[4] = {w0.x, w0.y, w0.z, w0.w}, a1[4] = {w1.x, w1.y, w1.z, w1.w};
#pragma unroll
        for (int G = 0; G < 4; ++G) {
            uint32_t ar[4], a8[4];
            unpack_w4(kc, a0[G], ar);
            unpack_w4(kc, a1[G], a8);
            step(G, ar[0], ar[1], ar[2], ar[3], a8[0], a8[1], a8[2], a8[3]);
        }
    } else if constexpr (BITS == 2) {
        const uint4 w = lds128(blob + slot16);
        const uint32_t a0[2] = {w.x, w.y}, a1[2] = {w.z, w.w};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t ar[8], a8[8];
            unpack_w2(kc, a0[h], ar);
            unpack_w2(kc, a1[h], a8);
#pragma unroll
            for (int gg = 0; gg < 2; ++gg)
                step(2 * h + gg, ar[4 * gg], ar[4 * gg + 1], ar[4 * gg + 2], ar[4 * gg + 3], a8[4 * gg], a8[4 * gg + 1], a8[4 * gg + 2], a8[4 * gg + 3]);
        }
    } else if constexpr (BITS == 8) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const uint4 w0 = lds128(blob + u * 512 + slot16), w1 = lds128(blob + 1024 + u * 512 + slot16);
            const uint32_t a0[4] = {w0.x, w0.y, w0.z, w0.w}, a1[4] = {w1.x, w1.y, w1.z, w1.w};
#pragma unroll
            for (int gg = 0; gg < 2; ++gg) {
                uint32_t ar[4], a8[4];
                unpack_w8(a0[2 * gg], a0[2 * gg + 1], ar);
                unpack_w8(a1[2 * gg], a1[2 * gg + 1], a8);
                step(2 * u + gg, ar[0], ar[1], ar[2], ar[3], a8[0], a8[1], a8[2], a8[3]);
            }
        }
    } else {
        const uint4 w0 = lds128(blob + slot16);
        const uint2 w1 = lds64(blob + 512 + (slot16 >> 1));
        uint32_t ar[16], a8[16];
        unpack_w3(kc, w0.x, w0.y, w0.z, ar);
        unpack_w3(kc, w0.w, w1.x, w1.y, a8);
#pragma unroll
        for (int G = 0; G < 4; ++G)
            step(G, ar[4 * G], ar[4 * G + 1], ar[4 * G + 2], ar[4 * G + 3], a8[4 * G], a8[4 * G + 1], a8[4 * G + 2], a8[4 * G + 3]);
    }
}

template <int BITS, int NT>
__device__ __forceinline__ void tile_mma(const GvConst& kc, uint32_t blob, int slot16, uint32_t xb, float (&acc)[NT][4]) {
    if constexpr (NT > 2) {
        tile_mma_wide<BITS, NT>(kc, blob, slot16, xb, acc);
        return;
    }
    uint4 b[NT][4];
#pragma unroll
    for (int G = 0; G < 4; ++G)
#pragma unroll
        for (int tb = 0; tb < NT; ++tb) b[tb][G] = lds128(xb + ((tb * 4 + G) << 9));
    if constexpr (BITS == 4) {
        const uint4 w0 = lds128(blob + slot16), w1 = lds128(blob + 512 + slot16);
        const uint32_t a0[4] = {w0.x, w0.y, w0.z, w0.w}, a1[4] = {w1.x, w1.y, w1.z, w1.w};
#pragma unroll
        for (int G = 0; G < 4; ++G) {
            uint32_t ar[4], a8[4];
            unpack_w4(kc, a0[G], ar);
            unpack_w4(kc, a1[G], a8);
#pragma unroll
            for (int tb = 0; tb < NT; ++tb) {
                mma_f16(acc[tb], ar[0], a8[0], ar[1], a8[1], b[tb][G].x, b[tb][G].y);
                mma_f16(acc[tb], ar[2], a8[2], ar[3], a8[3], b[tb][G].z, b[tb][G].w);
            }
        }
    } else if constexpr (BITS == 2) {
        // one 16-byte slot: {row g: chunks 0,1 | chunks 2,3 | row g + 8: chunks 0,1 | chunks 2,3}
        const uint4 w = lds128(blob + slot16);
        const uint32_t a0[2] = {w.x, w.y}, a1[2] = {w.z, w.w};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t ar[8], a8[8];
            unpack_w2(kc, a0[h], ar);
            unpack_w2(kc, a1[h], a8);
#pragma unroll
            for (int gg = 0; gg < 2; ++gg) {
#pragma unroll
                for (int tb = 0; tb < NT; ++tb) {
                    mma_f16(acc[tb], ar[4 * gg], a8[4 * gg], ar[4 * gg + 1], a8[4 * gg + 1], b[tb][2 * h + gg].x, b[tb][2 * h + gg].y);
                    mma_f16(acc[tb], ar[4 * gg + 2], a8[4 * gg + 2], ar[4 * gg + 3], a8[4 * gg + 3], b[tb][2 * h + gg].z, b[tb][2 * h + gg].w);
                }
            }
        }
    } else if constexpr (BITS == 8) {
        // 512-byte blocks of the blob: {row g: chunks 0,1}, {row g: chunks 2,3}, {row g + 8: chunks 0,1}, {row g + 8: chunks 2,3}
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const uint4 w0 = lds128(blob + u * 512 + slot16), w1 = lds128(blob + 1024 + u * 512 + slot16);
            const uint32_t a0[4] = {w0.x, w0.y, w0.z, w0.w}, a1[4] = {w1.x, w1.y, w1.z, w1.w};
#pragma unroll
            for (int gg = 0; gg < 2; ++gg) {
                uint32_t ar[4], a8[4];
                unpack_w8(a0[2 * gg], a0[2 * gg + 1], ar);
                unpack_w8(a1[2 * gg], a1[2 * gg + 1], a8);
#pragma unroll
                for (int tb = 0; tb < NT; ++tb) {
                    mma_f16(acc[tb], ar[0], a8[0], ar[1], a8[1], b[tb][2 * u + gg].x, b[tb][2 * u + gg].y);
                    mma_f16(acc[tb], ar[2], a8[2], ar[3], a8[3], b[tb][2 * u + gg].z, b[tb][2 * u + gg].w);
                }
            }
        }
    } else {
        const uint4 w0 = lds128(blob + slot16);
        const uint2 w1 = lds64(blob + 512 + (slot16 >> 1));
        uint32_t ar[16], a8[16];
        unpack_w3(kc, w0.x, w0.y, w0.z, ar);
        unpack_w3(kc, w0.w, w1.x, w1.y, a8);
#pragma unroll
        for (int G = 0; G < 4; ++G) {
#pragma unroll
            for (int tb = 0; tb < NT; ++tb) {
                mma_f16(acc[tb], ar[4 * G], a8[4 * G], ar[4 * G + 1], a8[4 * G + 1], b[tb][G].x, b[tb][G].y);
                mma_f16(acc[tb], ar[4 * G + 2], a8[4 * G + 2], ar[4 * G + 3], a8[4 * G + 3], b[tb][G].z, b[tb][G].w);
            }
        }
    }
}

// ---------------------------------------------------------------------------- the kernel
// NTMAX: token blocks of 8 rows an expert may get: 2 (batches of at most 16 rows), or 4 (at most 32 rows; its own
// instantiation, so that the common one keeps its registers)
template <bool FUSED, int NTMAX>
__global__ void __launch_bounds__(GV_THREADS, 1) qgemm_decode_kernel(const __grid_constant__ GvParams p) {
    using L = GvSmem<FUSED>;
    static_assert(NTMAX == 2 || (NTMAX == 4 && !FUSED), "gated pairs and residuals exist for batches of at most 16 rows");
    constexpr int SLOT_FLOATS = gv_slot_floats(NTMAX);
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_wfull = sbase + L::bar_off, bar_wempty = bar_wfull + 8 * GV_MAX_STAGES;
    const uint32_t bar_xfull = bar_wempty + 8 * GV_MAX_STAGES, bar_xempty = bar_xfull + 16;
    int* s_off = reinterpret_cast<int*>(smem + L::off_off);
    int* s_perm = reinterpret_cast<int*>(smem + L::perm_off);
    int* s_pair = reinterpret_cast<int*>(smem + L::pair_off);
    long long* s_base = reinterpret_cast<long long*>(smem + L::base_off);
    long long* s_C = reinterpret_cast<long long*>(smem + L::misc_off);
    int* s_G = reinterpret_cast<int*>(smem + L::misc_off + 8);
    int* s_geom = reinterpret_cast<int*>(smem + L::misc_off + 12);          // {stages, stage bytes}
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::misc_off + 20);
    ChunkDesc* s_desc = reinterpret_cast<ChunkDesc*>(smem + L::desc_off);
    const PairS* s_ps = reinterpret_cast<const PairS*>(smem + L::ps_off);

    // ---- prologue: nothing here depends on the previous kernel in the stream
    if (tid < p.P * 12) reinterpret_cast<int*>(smem + L::ps_off)[tid] = reinterpret_cast<const int*>(p.ps)[tid];
    if (tid == 0) {
        for (int i = 0; i < GV_MAX_STAGES; ++i) { mbar_init(bar_wfull + 8 * i, 1); mbar_init(bar_wempty + 8 * i, GV_CONS); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar_xfull + 8 * i, GV_SERV * 32); mbar_init(bar_xempty + 8 * i, GV_CONS); }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // ---- the work split, by warp 0: lane v works out pair v from the offset table (read past L1: the table may be
    // rewritten by the previous kernel between the two reads below)
    auto work_split = [&]() {
        const int v = lane;
        long long cost = 0;
        int TT = 0, wv = 1;
        {
            const PairS q = p.ps[v < p.P ? v : 0];
            const int rows = __ldcg(p.offsets + q.rexp + 1) - __ldcg(p.offsets + q.rexp);
            wv = q.w;
            TT = (v < p.P && rows > 0) ? ((FUSED && q.gated) ? q.NT1 : (q.NT1 + 1) >> 1) * q.KB : 0;
            cost = (long long)TT * wv;
        }
        long long incl = cost;
        int wmax = TT > 0 ? wv : 1;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const long long o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
            wmax = max(wmax, __shfl_xor_sync(0xffffffffu, wmax, d));
        }
        const long long C = __shfl_sync(0xffffffffu, incl, 31);
        const long long base = incl - cost;
        // every CTA's share holds at least one super-tile start
        const long long Gl = p.small ? (long long)((unsigned)C / (unsigned)wmax) : C / wmax;
        const int G = (int)(Gl < (long long)gridDim.x ? Gl : (long long)gridDim.x);
        int tb = 0, te = 0, str = 0;
        if (v < p.P) {
            if (TT > 0 && (int)blockIdx.x < G) {
                const long long den = (long long)wv * G;
                const long long n0 = (long long)blockIdx.x * C - base * G, n1 = (long long)(blockIdx.x + 1) * C - base * G;
                long long t0, t1;
                if (p.small) {                                  // the same quotients from 32-bit divisions
                    const unsigned d32 = (unsigned)den;
                    t0 = n0 <= 0 ? 0 : (long long)(((unsigned)n0 + d32 - 1) / d32);
                    t1 = n1 <= 0 ? 0 : (long long)(((unsigned)n1 + d32 - 1) / d32);
                } else {
                    t0 = n0 <= 0 ? 0 : (n0 + den - 1) / den;
                    t1 = n1 <= 0 ? 0 : (n1 + den - 1) / den;
                }
                tb = (int)(t0 > TT ? TT : t0);
                te = (int)(t1 > TT ? TT : t1);
            }
            s_pair[2 * v] = tb;
            s_pair[2 * v + 1] = te;
            s_base[v] = base;
            if (te > tb) str = p.ps[v].stride;
        }
        // ring geometry: a stage holds two of the largest packed tiles this CTA will see
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) str = max(str, __shfl_xor_sync(0xffffffffu, str, d));
        if (lane == 0) {
            const int stage_bytes = 2 * ((max(str, 128) + 127) & ~127);
            *s_C = C; *s_G = G;
            s_geom[0] = min(GV_MAX_STAGES, L::ring_bytes / stage_bytes);
            s_geom[1] = stage_bytes;
        }
    };
    // A guess at the split from whatever the offset table holds before the previous kernel is known to have finished
    // (in a block's later launches it is final already), used ONLY to ask L2 for the first packed tiles this CTA would
    // stream: a CTA that starts while the previous kernel's last CTAs are still running spends the wait pulling its
    // weights out of HBM.  A wrong guess costs some prefetched lines; every address lies inside the pair's tile array.
    int guess_off = 0, guess_last = 0;
    if (warp == 0) {
        guess_off = lane <= p.R ? __ldcg(p.offsets + lane) : 0;
        guess_last = p.R >= 32 ? __ldcg(p.offsets + p.R) : 0;
        work_split();
        __syncwarp();
        if (lane == 0) {
            GvWalk wk;
            wk.start();
            bool changed;
            int left = GV_PREFETCH_TILES;
            while (left > 0 && wk.next(s_pair, p.ps, p.P, changed)) {
                const int v = wk.v, n = min(wk.run(), left);
                const PairS q = p.ps[v];
                const bool gated = FUSED && q.gated;
                const int nt = gated ? wk.nt2 : 2 * wk.nt2;
                const uint8_t* a = p.ex[v].tiles + ((size_t)nt * wk.KB + wk.kb) * q.stride;
                const uint8_t* b2 = gated ? p.tiles2[v] + ((size_t)nt * wk.KB + wk.kb) * q.stride
                                          : (nt + 1 < q.NT1 ? a + (size_t)wk.KB * q.stride : nullptr);
                // the run's tiles are contiguous: one request per 128-channel tile row
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a), "r"(n * q.stride) : "memory");
                if (b2) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(b2), "r"(n * q.stride) : "memory");
                left -= n;
            }
        }
    }
    // from here on the previous kernel's results are needed (sort tables, activations, workspace)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid >= 32 && tid <= 32 + p.R) s_off[tid - 32] = __ldcg(p.offsets + tid - 32);
    if (tid >= 64 && tid < 64 + 8 * NTMAX) s_perm[tid - 64] = tid - 64 < p.M ? p.perm[tid - 64] : 0;
    if (warp == 0) {
        const int my_off = lane <= p.R ? __ldcg(p.offsets + lane) : 0;
        const int my_last = p.R >= 32 ? __ldcg(p.offsets + p.R) : 0;
        if (!__all_sync(0xffffffffu, my_off == guess_off && my_last == guess_last)) work_split();   // (else the guess was the split)
    }
    __syncthreads();
    const int nstg = s_geom[0], stage_bytes = s_geom[1];

    // ---- staging of one chunk of token rows by `nthr` threads (a multiple of 32; this one is number st of them, st % 32 its
    // lane).  A row tile -- the 128 values X[row m][k-block] -- is sixteen 16-byte fetches, each converted to four fp16
    // pairs in MMA fragment order, plus the row tile's sums.  The service warps give a thread whole row tiles (eight
    // fetches in flight, no exchange between threads); the first chunk, staged by all warps together, gives it one
    // 32-value group of a row tile (one fetch latency; the sums are added up over four lanes).  The caller's walk is
    // advanced past the chunk.  Returns false when there was no chunk left (an invalid descriptor has been written).
    auto stage_chunk = [&](auto parts_tag, GvWalk& wk, int& kbc, bool& more, int n, int nthr, int st) -> bool {
        constexpr int PARTS = decltype(parts_tag)::value;       // threads per row tile: 1, or 4 (one 32-value group each)
        const int buf = n & 1;
        ChunkDesc* d = s_desc + buf;
        if (!more) {
            if (st == 0) d->valid = 0;
            return false;
        }
        const int v = wk.v;
        const int row0 = s_off[s_ps[v].rexp], rows = s_off[s_ps[v].rexp + 1] - row0;
        const int ntl = (NTMAX > 2 && rows > 16) ? 2 : (rows > 8 ? 1 : 0), NT = 1 << ntl;      // token blocks: 1, 2 or 4
        const int kb1 = wk.kb + wk.run();
        const int nkb = min(GV_CHUNK_KB >> ntl, kb1 - kbc);
        if (st == 0) { d->v = v; d->nt2 = wk.nt2; d->kbc = kbc; d->nkb = nkb; d->kb0 = wk.kb; d->kb1 = kb1; d->valid = 1; }
        const int bits = s_ps[v].bits, K = s_ps[v].K;
        const float fold = s_ps[v].has_zeros ? 0.f : (float)(1 << (bits - 1));   // a constant zero-point goes into the sums
        const uint32_t xbuf = sbase + L::x_off + buf * GV_XBUF;
        float* sbuf = reinterpret_cast<float*>(smem + L::s_off + buf * GV_SBUF);
        // (the format's scale exponents are compile-time constants: one instantiation of the loop per code width)
        auto stage_units = [&](auto bits_tag) {
            // one 16-byte fetch (chunk a = 4G + q of the k-block: k = 32G + 8q ..) -> four fp16 pairs in MMA fragment order at
            // [slab][G][lane = 4 mm + q]; the pair sums go into the group's partial sums
            auto convert = [&](const uint4& dat, int a, uint32_t xdst, float& S0, float& S1) {
                const int G = a >> 2, q = a & 3;
                const uint32_t w[4] = {dat.x, dat.y, dat.z, dat.w};
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    // pair p = 4G + j of the piece: scaled by sigma = 2^-e, e fixed by the format
                    constexpr int BITS = decltype(bits_tag)::value;
                    const int e = sigma_shift(BITS, 4 * G + j);
                    const float lo = __uint_as_float(w[j] << 16), hi = __uint_as_float(w[j] & 0xFFFF0000u);
                    const float sum = lo + hi;
                    S0 += sum;
                    S1 = fmaf(__int_as_float((127 - e) << 23), sum, S1);
                    __half2 hh = __floats2half2_rn(lo, hi);
                    const uint32_t sg = (uint32_t)((15 - e) << 10) * 0x00010001u;
                    hh = __hmul2(hh, *reinterpret_cast<const __half2*>(&sg));
                    o[j] = *reinterpret_cast<uint32_t*>(&hh);
                }
                sts128(xdst + (G << 9) + (q << 4), o[0], o[1], o[2], o[3]);
            };
            // row tiles of the chunk: rt = slab * 8 + mm, slab = k-block * NT + token block.  The sums of a row tile are
            // (g0 + g1) + (g2 + g3) over its four 32-value groups, whoever stages it.
            const int units = nkb * NT * 8 * PARTS;
            for (int u0 = st & ~31; u0 < units; u0 += nthr) {
                const int unit = u0 + (st & 31);
                const bool live = unit < units;
                const int rt = unit / PARTS, part = unit % PARTS;
                const int slab = rt >> 3, mm = rt & 7;
                const int kbl = slab >> ntl, m = (slab & (NT - 1)) * 8 + mm;
                const int k0 = (kbc + kbl) * 128;
                const uint16_t* src = live && m < rows ? p.X[v] + (size_t)s_perm[row0 + m] * K + k0 : nullptr;
                const uint32_t xdst = xbuf + (slab << 11) + (mm << 6);
                float S0, S1;
                if constexpr (PARTS == 4) {
                    uint4 data[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int a = 4 * part + i;
                        data[i] = make_uint4(0, 0, 0, 0);
                        if (src != nullptr && k0 + a * 8 < K) data[i] = __ldg(reinterpret_cast<const uint4*>(src + a * 8));
                    }
                    S0 = 0.f; S1 = 0.f;
                    if (live) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) convert(data[i], 4 * part + i, xdst, S0, S1);
                    }
                    S0 += __shfl_xor_sync(0xffffffffu, S0, 1);
                    S1 += __shfl_xor_sync(0xffffffffu, S1, 1);
                    S0 += __shfl_xor_sync(0xffffffffu, S0, 2);
                    S1 += __shfl_xor_sync(0xffffffffu, S1, 2);
                } else {
                    float g0[4] = {0.f, 0.f, 0.f, 0.f}, g1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        uint4 data[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int a = 8 * h + i;
                            data[i] = make_uint4(0, 0, 0, 0);
                            if (src != nullptr && k0 + a * 8 < K) data[i] = __ldg(reinterpret_cast<const uint4*>(src + a * 8));
                        }
                        if (live) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) convert(data[i], 8 * h + i, xdst, g0[2 * h + (i >> 2)], g1[2 * h + (i >> 2)]);
                        }
                    }
                    S0 = (g0[0] + g0[1]) + (g0[2] + g0[3]);
                    S1 = (g1[0] + g1[1]) + (g1[2] + g1[3]);
                }
                // sums at [slab][t = mm / 2][4]
                if (live && part == 0) {
                    float* S = sbuf + slab * 16 + (mm >> 1) * 4 + (mm & 1);
                    S[0] = fmaf(-1024.f, S1, -fold * S0);              // what the accumulator starts from
                    S[2] = S0;
                }
            }
        };
        switch (bits) {
            case 8: stage_units(std::integral_constant<int, 8>{}); break;
            case 4: stage_units(std::integral_constant<int, 4>{}); break;
            case 3: stage_units(std::integral_constant<int, 3>{}); break;
            default: stage_units(std::integral_constant<int, 2>{}); break;
        }
        kbc += nkb;
        if (kbc >= kb1) {
            bool changed;
            more = wk.next(s_pair, s_ps, p.P, changed);
            kbc = more ? wk.kb : 0;
        }
        return true;
    };
    // the first chunk is staged by the consumer and service warps together: one fetch latency instead of many
    GvWalk swk;
    swk.start();
    bool s_changed, s_more = swk.next(s_pair, s_ps, p.P, s_changed);
    int s_kbc = s_more ? swk.kb : 0;
    if (warp < GV_CONS + GV_SERV) {
        stage_chunk(std::integral_constant<int, 4>{}, swk, s_kbc, s_more, 0, (GV_CONS + GV_SERV) * 32, tid);
        asm volatile("bar.sync 1, %0;" ::"n"((GV_CONS + GV_SERV) * 32) : "memory");   // (the producer is already streaming)
    }

    if (warp == GV_CONS + GV_SERV) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            const uint64_t once = l2_policy_evict_first();
            GvWalk wk;
            wk.start();
            Ring ring;
            bool changed, ok = true;
            int issued = 0;
            while (ok && wk.next(s_pair, s_ps, p.P, changed)) {
                const int v = wk.v, n = wk.run();
                const uint32_t stride = (uint32_t)s_ps[v].stride;
                const bool gated = FUSED && s_ps[v].gated;
                const int nt = gated ? wk.nt2 : 2 * wk.nt2;
                const bool two = gated || nt + 1 < s_ps[v].NT1;
                const uint8_t* a = p.ex[v].tiles + ((size_t)nt * wk.KB + wk.kb) * stride;
                const uint8_t* b = gated ? p.tiles2[v] + ((size_t)nt * wk.KB + wk.kb) * stride : a + (size_t)wk.KB * stride;
                for (int i = 0; i < n; ++i) {
                    // Ramp-up: when all CTAs ask for a full ring at once, a CTA's first tile queues behind everybody's
                    // ninth; so the first two stages go out alone and the rest follows once the first has landed.
                    if (issued == 2 && !mbar_wait(bar_wfull, 0u, s_abort, p.status)) { ok = false; break; }
                    ++issued;
                    if (!mbar_wait(bar_wempty + 8 * ring.stage, ring.phase ^ 1u, s_abort, p.status)) { ok = false; break; }
                    const uint32_t full = bar_wfull + 8 * ring.stage;
                    const uint32_t dst = sbase + L::ring_off + ring.stage * stage_bytes;
                    mbar_expect_tx(full, two ? 2 * stride : stride);
                    bulk_load_once(dst, a, stride, full, once);
                    if (two) bulk_load_once(dst + (stage_bytes >> 1), b, stride, full, once);
                    a += stride; b += stride;
                    ring.advance(nstg);
                }
            }
        }
    } else if (warp >= GV_CONS) {
        // ------------------------------------------------------------------ service warps: token rows, one chunk ahead
        const int st = tid - GV_CONS * 32;
        for (int n = 1;; ++n) {
            const int buf = n & 1;
            if (n >= 2 && !__all_sync(0xffffffffu, mbar_wait(bar_xempty + 8 * buf, (uint32_t)((n >> 1) - 1) & 1u, s_abort, p.status))) break;
            const bool staged = stage_chunk(std::integral_constant<int, 1>{}, swk, s_kbc, s_more, n, GV_SERV * 32, st);
            mbar_arrive(bar_xfull + 8 * buf);
            if (!staged) break;
        }
    } else {
        // ------------------------------------------------------------------ consumer warps
        const int g = lane >> 2, t = lane & 3;
        const int half = warp >> 3, blob = warp & 7;
        const int slot16 = (t * 8 + (g ^ (2 * t))) * 16;          // this lane's 16-byte slot inside a 512-byte half blob
        const uint32_t tile_base = sbase + L::ring_off + half * (stage_bytes >> 1);
        Ring ring;
        float fin[4 * NTMAX];                             // the running sums of the current piece: [token block][4]
#pragma unroll
        for (int i = 0; i < 4 * NTMAX; ++i) fin[i] = 0.f;
        float sc_r = 0.f, sc_r8 = 0.f, z_r = 0.f, z_r8 = 0.f;     // per-channel experts: scale / zero-point of rows g, g + 8
        bool ok = true;

        // One chunk of k-blocks of one piece, for a format fixed at compile time.
        auto run_chunk = [&](auto tag, int nkb, int buf, bool active) {
            constexpr int BITS = decltype(tag)::bits, NT = decltype(tag)::nt;
            constexpr bool GROUPED = decltype(tag)::grouped, ASYM = decltype(tag)::asym;
            GvConst kc;
            kc.template init<BITS>();
            const uint32_t xb0 = sbase + L::x_off + buf * GV_XBUF + lane * 16;
            const float4* sS = reinterpret_cast<const float4*>(smem + L::s_off + buf * GV_SBUF) + t;
            const uint32_t blob_off = blob * (BITS * 256);
            const uint32_t meta_off = moqe_tile_bytes(BITS) + (blob * 16 + g) * 2;
#pragma unroll 1
            for (int kbl = 0; kbl < nkb; ++kbl) {
                if (!__all_sync(0xffffffffu, mbar_wait_short(bar_wfull + 8 * ring.stage, ring.phase, s_abort, p.status))) { ok = false; return; }
                if (active) {
                    const uint32_t tile = tile_base + ring.stage * stage_bytes;
                    float acc[NT][4], S0[NT][2];
#pragma unroll
                    for (int tb = 0; tb < NT; ++tb) {
                        const float4 sv = sS[(kbl * NT + tb) * 4];
                        acc[tb][0] = acc[tb][2] = sv.x;
                        acc[tb][1] = acc[tb][3] = sv.y;
                        S0[tb][0] = sv.z;
                        S0[tb][1] = sv.w;
                    }
                    float s0 = sc_r, s8 = sc_r8, z0 = z_r, z8 = z_r8;
                    if constexpr (GROUPED) {
                        const uint32_t meta = tile + meta_off;
                        s0 = __half2float(__ushort_as_half((unsigned short)lds16(meta)));
                        s8 = __half2float(__ushort_as_half((unsigned short)lds16(meta + 16)));
                        if constexpr (ASYM) {
                            z0 = __uint_as_float(lds16(meta + 256) << 16);
                            z8 = __uint_as_float(lds16(meta + 256 + 16) << 16);
                        }
                    }
                    tile_mma<BITS, NT>(kc, tile + blob_off, slot16, xb0 + ((kbl * NT * 4) << 9), acc);
                    // the k-block is complete: scale and add
#pragma unroll
                    for (int tb = 0; tb < NT; ++tb) {
                        if constexpr (ASYM) {
                            fin[4 * tb + 0] = fmaf(s0, fmaf(-z0, S0[tb][0], acc[tb][0]), fin[4 * tb + 0]);
                            fin[4 * tb + 1] = fmaf(s0, fmaf(-z0, S0[tb][1], acc[tb][1]), fin[4 * tb + 1]);
                            fin[4 * tb + 2] = fmaf(s8, fmaf(-z8, S0[tb][0], acc[tb][2]), fin[4 * tb + 2]);
                            fin[4 * tb + 3] = fmaf(s8, fmaf(-z8, S0[tb][1], acc[tb][3]), fin[4 * tb + 3]);
                        } else {
                            fin[4 * tb + 0] = fmaf(s0, acc[tb][0], fin[4 * tb + 0]);
                            fin[4 * tb + 1] = fmaf(s0, acc[tb][1], fin[4 * tb + 1]);
                            fin[4 * tb + 2] = fmaf(s8, acc[tb][2], fin[4 * tb + 2]);
                            fin[4 * tb + 3] = fmaf(s8, acc[tb][3], fin[4 * tb + 3]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_wempty + 8 * ring.stage);
                ring.advance(nstg);
            }
        };

        for (int n = 0; ok; ++n) {
            const int buf = n & 1;
            if (n > 0 && !__all_sync(0xffffffffu, mbar_wait(bar_xfull + 8 * buf, (uint32_t)((n - 1) >> 1) & 1u, s_abort, p.status))) break;
            const ChunkDesc* d = s_desc + buf;
            if (!d->valid) break;
            const int v = d->v, nt2 = d->nt2, kbc = d->kbc, nkb = d->nkb, kb0 = d->kb0, kb1 = d->kb1;
            const int row0 = s_off[s_ps[v].rexp], rows = s_off[s_ps[v].rexp + 1] - row0;
            const int bits = s_ps[v].bits, group = s_ps[v].group, has_zeros = s_ps[v].has_zeros;
            const bool gated = FUSED && s_ps[v].gated;
            const int nt = gated ? nt2 : 2 * nt2 + half;
            const bool active = nt < s_ps[v].NT1;
            const int n_r = nt * 128 + blob * 16 + g;
            if (kbc == kb0) {
#pragma unroll
                for (int i = 0; i < 4 * NTMAX; ++i) fin[i] = 0.f;
                if (group == 0 && active) {
                    const __half* sp = gated && half ? p.scales_pc2[v] : p.ex[v].scales_pc;
                    sc_r = __half2float(sp[n_r]);
                    sc_r8 = __half2float(sp[n_r + 8]);
                    if (has_zeros) {
                        const __nv_bfloat16* zp = gated && half ? p.zeros_pc2[v] : p.ex[v].zeros_pc;
                        z_r = __bfloat162float(zp[n_r]);
                        z_r8 = __bfloat162float(zp[n_r + 8]);
                    }
                }
            }
            // dispatch on the format (uniform over the CTA)
            const int nti = (NTMAX > 2 && rows > 16) ? 2 : (rows > 8 ? 1 : 0);                  // 1, 2 or 4 token blocks
            const int fmt = (bits == 4 ? 0 : (bits == 8 ? 1 : (bits == 3 ? 2 : 3))) * 12 + nti * 4 + (group != 0 ? 2 : 0) + (has_zeros ? 1 : 0);
            switch (fmt) {
#define GV_CASE(B, BI, NTI, GR, AS) \
                case BI * 12 + NTI * 4 + GR * 2 + AS: \
                    if constexpr ((1 << NTI) <= NTMAX) run_chunk(GvTag<B, (1 << NTI), GR != 0, AS != 0>{}, nkb, buf, active); \
                    break;
#define GV_CASES(B, BI) GV_CASE(B, BI, 0, 0, 0) GV_CASE(B, BI, 0, 0, 1) GV_CASE(B, BI, 0, 1, 0) GV_CASE(B, BI, 0, 1, 1) \
                        GV_CASE(B, BI, 1, 0, 0) GV_CASE(B, BI, 1, 0, 1) GV_CASE(B, BI, 1, 1, 0) GV_CASE(B, BI, 1, 1, 1) \
                        GV_CASE(B, BI, 2, 0, 0) GV_CASE(B, BI, 2, 0, 1) GV_CASE(B, BI, 2, 1, 0) GV_CASE(B, BI, 2, 1, 1)
                GV_CASES(4, 0)
                GV_CASES(8, 1)
                GV_CASES(3, 2)
                GV_CASES(2, 3)
#undef GV_CASES
#undef GV_CASE
                default: break;
            }
            if (!ok) break;

            if (kbc + nkb == kb1 && active) {
                // ---- the piece is complete
                const int NT = 1 << nti;
                const int KB = s_ps[v].KB, N = s_ps[v].N;
                uint16_t* Y = p.Y[v];
                const uint16_t* R = FUSED ? p.Res[v] : nullptr;
                auto store_rows = [&]() {
#pragma unroll
                    for (int tb = 0; tb < NTMAX; ++tb) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int m = 8 * tb + 2 * t + (j & 1), nn = n_r + (j >> 1) * 8;
                            if (tb < NT && m < rows && nn < N) {
                                const size_t at = (size_t)s_perm[row0 + m] * N + nn;
                                float y = fin[4 * tb + j];
                                if (R) y += __uint_as_float((uint32_t)R[at] << 16);
                                Y[at] = __bfloat16_as_ushort(__float2bfloat16_rn(y));
                            }
                        }
                    }
                };
                // gated pair: fin <- silu(fin) * other, the second expert's product of the same channels and rows
                auto gate_with = [&](const float (&other)[4 * NTMAX]) {
#pragma unroll
                    for (int i = 0; i < 4 * NTMAX; ++i) fin[i] = fin[i] / (1.f + expf(-fin[i])) * other[i];
                };
                float* xchg = reinterpret_cast<float*>(smem + L::xchg_off) + blob * 256 + lane;
                if (kb0 == 0 && kb1 == KB) {
                    if (FUSED && gated) {
                        // warps w and w + 8 hold the two products of the same channels: hand the second to the first
                        if (half == 1) {
#pragma unroll
                            for (int i = 0; i < 4 * NTMAX; ++i) xchg[i * 32] = fin[i];
                        }
                        asm volatile("bar.sync %0, 64;" ::"r"(2 + blob) : "memory");
                        if (half == 0) {
                            float other[4 * NTMAX];
#pragma unroll
                            for (int i = 0; i < 4 * NTMAX; ++i) other[i] = xchg[i * 32];
                            gate_with(other);
                            store_rows();
                        }
                        asm volatile("bar.sync %0, 64;" ::"r"(2 + blob) : "memory");     // the buffer may be written again
                    } else {
                        store_rows();
                    }
                } else {
                    // part of a segment: park this warp's sums, announce, and add everything up if this was the last arrival
                    // (for a gated pair the two warps of a blob share one counter and whoever is last finishes both products)
                    const long long C = *s_C, base = s_base[v];
                    const int G = *s_G, wv = s_ps[v].w;
                    const int c_a = (int)(((base + (long long)(nt2 * KB) * wv) * G) / C);
                    const int c_b = (int)(((base + (long long)(nt2 * KB + KB - 1) * wv) * G) / C);
                    float* slot = p.partials + (size_t)(2 * blockIdx.x + (kb0 == 0 ? 1 : 0)) * SLOT_FLOATS;
#pragma unroll
                    for (int tb = 0; tb < NTMAX; ++tb)
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (tb < NT) __stcg(slot + ((warp * NTMAX + tb) * 4 + j) * 32 + lane, fin[4 * tb + j]);
                    __syncwarp();
                    unsigned* counter = p.counters + c_a * GV_CONS + (gated ? blob : warp);
                    const unsigned last = (unsigned)(gated ? 2 * (c_b - c_a) + 1 : c_b - c_a);
                    unsigned arrived = 0;
                    // one acquire-release increment: the release side publishes the warp's parked sums (ordered before it
                    // by the warp barrier above), the acquire side lets the last arriver read everybody else's
                    if (lane == 0) asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(arrived) : "l"(counter) : "memory");
                    arrived = __shfl_sync(0xffffffffu, arrived, 0);
                    if (arrived == last) {
                        __syncwarp();
                        auto gather = [&](int wsrc, float (&dst)[4 * NTMAX]) {
#pragma unroll
                            for (int i = 0; i < 4 * NTMAX; ++i) dst[i] = 0.f;
                            // several CTAs' sums are fetched together (one round trip), then added in CTA order
                            constexpr int GB = NTMAX == 2 ? 4 : 2;
                            for (int c0 = c_a; c0 <= c_b; c0 += GB) {
                                float part[GB][4 * NTMAX];
#pragma unroll
                                for (int u = 0; u < GB; ++u) {
                                    const int c = c0 + u;
                                    const float* src = p.partials + (size_t)(2 * c + (c == c_a ? 1 : 0)) * SLOT_FLOATS;
#pragma unroll
                                    for (int tb = 0; tb < NTMAX; ++tb)
#pragma unroll
                                        for (int j = 0; j < 4; ++j)
                                            part[u][4 * tb + j] = (c <= c_b && tb < NT) ? __ldcg(src + ((wsrc * NTMAX + tb) * 4 + j) * 32 + lane) : 0.f;
                                }
#pragma unroll
                                for (int u = 0; u < GB; ++u)
#pragma unroll
                                    for (int i = 0; i < 4 * NTMAX; ++i) dst[i] += part[u][i];
                            }
                        };
                        if (FUSED && gated) {
                            float other[4 * NTMAX];
                            gather(blob, fin);
                            gather(blob + 8, other);
                            gate_with(other);
                        } else {
                            gather(warp, fin);
                        }
                        store_rows();
                        if (lane == 0) *counter = 0u;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_xempty + 8 * buf);
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncthreads();
    if (*s_abort) {
        // let bulk copies that may still be in flight land before the shared memory is released
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
    }
}

int dec_sm_count() {
    int dev = 0, n = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n > 0 ? n : 148;
}

// relative cost of one super-tile in the work split, by code width (measured: a 3-bit super-tile takes the consumers
// about a tenth longer than a 4-bit one, an 8-bit one lies between -- its copies are twice as large)
int g_dec_cost[9] = {0, 0, 20, 22, 20, 0, 0, 0, 21};

bool dec_formats_ok(const moqe_expert* const* ex, int n) {
    for (int v = 0; v < n; ++v) {
        if (ex[v]->bits != 2 && ex[v]->bits != 3 && ex[v]->bits != 4 && ex[v]->bits != 8) return false;
        if (ex[v]->group != 0 && (ex[v]->group < 128 || ex[v]->group % 128 != 0)) return false;
    }
    return true;
}

}  // namespace

void decode_set_tile_cost(int bits, int cost) { if (bits >= 0 && bits <= 8 && cost > 0) g_dec_cost[bits] = cost; }

bool decode_supported_multi(int M, const moqe_expert* const* ex, int nl, int E) {
    return M <= DECODE_MAX_ROWS && nl >= 1 && nl * E <= MOQE_MAX_EXPERTS && dec_formats_ok(ex, nl * E);
}

size_t decode_zero_bytes(int M) { return M > DECODE_MAX_ROWS ? 0 : (size_t)GV_MAX_GRID * GV_CONS * sizeof(uint32_t); }

size_t decode_workspace_bytes(int M) {
    if (M > DECODE_MAX_ROWS) return 0;
    return (decode_zero_bytes(M) + 255) / 256 * 256 + (size_t)GV_MAX_GRID * 2 * gv_slot_floats(M > 16 ? 4 : 2) * sizeof(float);
}

// nl layers that share the routing; ex[l * E + e] = expert e of layer l; X[l] / Y[l] the layer's input / output
moqe_status launch_qgemm_decode_multi(const void* const* X, int M, int nl, const moqe_expert* const* ex, int E,
                                    void* const* Y, const int32_t* perm, const int32_t* offsets, void* ws,
                                    size_t ws_bytes, cudaStream_t st) {
    return launch_qgemm_decode_ext(X, M, nl, ex, nullptr, E, Y, nullptr, perm, offsets, ws, ws_bytes, st);
}

// ex2 (or nullptr): per (layer, expert) the second expert of a gated pair, Y = silu(X.W1^T) * (X.W2^T), or nullptr for a
// plain layer; R (or nullptr): per layer a residual [M][N] added before the rounding, or nullptr
moqe_status launch_qgemm_decode_ext(const void* const* X, int M, int nl, const moqe_expert* const* ex,
                                  const moqe_expert* const* ex2, int E, void* const* Y, const void* const* R,
                                  const int32_t* perm, const int32_t* offsets, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (M == 0) return MOQE_OK;
    if (!decode_supported_multi(M, ex, nl, E)) return MOQE_ERR_UNSUPPORTED;
    if (ex2)
        for (int v = 0; v < nl * E; ++v)
            if (ex2[v] && (ex2[v]->N != ex[v]->N || ex2[v]->K != ex[v]->K || ex2[v]->bits != ex[v]->bits ||
                           ex2[v]->group != ex[v]->group || ex2[v]->sym != ex[v]->sym))
                return MOQE_ERR_MISMATCH;
    if (!ws || ws_bytes < decode_workspace_bytes(M)) return MOQE_ERR_WORKSPACE;
    GvParams p;
    long long total_cost = 0;                       // with every expert touched: an upper bound of what the kernel adds up
    for (int l = 0; l < nl; ++l)
        for (int e = 0; e < E; ++e) {
            const int v = l * E + e;
            p.ex[v] = ex[v]->dev();
            p.X[v] = (const uint16_t*)X[l];
            p.Y[v] = (uint16_t*)Y[l];
            const moqe_expert* second = ex2 ? ex2[v] : nullptr;
            PairS& q = p.ps[v];
            q.bits = p.ex[v].bits; q.group = p.ex[v].group; q.has_zeros = p.ex[v].has_zeros; q.stride = p.ex[v].tile_stride;
            q.N = ex[v]->N; q.K = ex[v]->K; q.KB = ex[v]->Kp / 128; q.NT1 = ex[v]->Np / 128;
            q.rexp = e;
            q.w = g_dec_cost[ex[v]->bits];
            q.gated = second ? 1 : 0;
            q.pad = 0;
            total_cost += (long long)(second ? q.NT1 : (q.NT1 + 1) / 2) * q.KB * q.w;
            p.tiles2[v] = second ? second->tiles : nullptr;
            p.scales_pc2[v] = second ? second->scales_pc : nullptr;
            p.zeros_pc2[v] = second ? second->zeros_pc : nullptr;
            p.Res[v] = R ? (const uint16_t*)R[l] : nullptr;
        }
    p.counters = (uint32_t*)ws;
    p.partials = (float*)((char*)ws + (decode_zero_bytes(M) + 255) / 256 * 256);
    p.perm = perm;
    p.offsets = offsets;
    p.M = M;
    p.R = E;
    p.P = nl * E;
    p.status = device_status_word();
    int grid = dec_sm_count();
    if (grid > GV_MAX_GRID) grid = GV_MAX_GRID;
    p.small = total_cost * (grid + 1) < (1ll << 31) ? 1 : 0;
    const bool fused = ex2 != nullptr || R != nullptr;
    if (fused && M > 16) return MOQE_ERR_UNSUPPORTED;     // gated pairs and residual adds: batches of at most 16 rows
    const int smem = fused ? GvSmem<true>::dyn_bytes : GvSmem<false>::dyn_bytes;
    auto kernel = fused ? qgemm_decode_kernel<true, 2> : (M > 16 ? qgemm_decode_kernel<false, 4> : qgemm_decode_kernel<false, 2>);
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (err == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid); cfg.blockDim = dim3(GV_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        err = cudaLaunchKernelEx(&cfg, kernel, p);
    }
    if (err != cudaSuccess) return MOQE_ERR_CUDA;
    count_launch();
    return cuda_ok(cudaGetLastError());
}

}  // namespace moqe
