// Routed dequant-GEMM for small batches (decode shapes): every touched expert's
// packed weights are streamed from HBM exactly once.
//
//   producer warp : cp.async.bulk copies whole packed 128x128-code tiles (6-16 KiB,
//                   contiguous in HBM), the expert's token rows for the same 128 k
//                   (gathered through `perm`: the fused permutation) and the tile's
//                   scales / zero-points into a ring of shared-memory stages, each
//                   guarded by a full/empty mbarrier pair.  Many stages are in flight
//                   per SM, which is what keeps HBM busy; no register is spent on it.
//   8 consumer    : warp w owns the 16 channels of blob w.  It reads its packed words
//   warps           with conflict-free 128-bit shared loads, unpacks them in registers
//                   to the exact integers (c - z) in bf16, and issues warp-level
//                   m16n8k16 tensor-core MMAs (weights = 16-row operand, up to 8 tokens
//                   per column block).  Group scales are applied in fp32 outside the
//                   MMA ("two-level accumulation"):
//                     Y[m][n] = sum_G s[n][G] * (sum_{k in G} X[m][k] * (c[n][k] - z[n][G]))
//                   so the tensor core only sees exactly representable operands.
//   work units    : (expert, 128-channel tile, K split), dealt round-robin to a
//                   persistent grid of 2 CTAs per SM; K is split so that units carry
//                   about equal bytes whatever the expert's bit-width, and the ring
//                   keeps filling across unit boundaries.  Split partials go to a
//                   workspace; the last CTA to arrive for a (tile, token chunk) adds
//                   them in fixed split order and writes bf16 rows straight to their
//                   original positions (fused un-permutation, deterministic result).
//
// CUDA cores could not keep up with HBM here (about 13e12 4-bit codes/s, each
// needing one FMA per token row), hence tensor-core MMAs even for 16 rows.
//
// Section 3.1 of the paper ("the activated quantization expert performs the
// inference on this sample") is the operation; the paper describes no kernel.
#include <type_traits>

#include "dequant.cuh"
#include "ptx.cuh"

namespace moqe {
namespace {

constexpr int CONSUMER_WARPS = 8;
constexpr int STREAM_THREADS = (CONSUMER_WARPS + 2) * 32;   // + one producer warp + one fix-up warp
constexpr int W_BYTES = 128 * 128 + 4 * 512;  // largest packed tile (W8 codes) + largest per-tile meta (4 groups, asymmetric)
constexpr int XROW = 320;                     // staged token row: 128 k of bf16 + pad; = 64 mod 128 (conflict-free LDS.128)
constexpr int OUT_STRIDE = 132;               // floats per staged output row
constexpr int MAX_STAGES = 12;
constexpr int SPLIT_MAX_ROWS = 64;            // K is split across CTAs only for batches this small

template <int NTMAX>
struct StreamSmem {
    static constexpr int T = 8 * NTMAX;                       // token rows per chunk
    // the ring: room for 4 (3 for 32-token chunks) stages of the largest tile; CTAs whose experts have
    // smaller tiles cut it into more, smaller stages (up to MAX_STAGES) to keep as many bytes in flight
    static constexpr int ring_bytes = (NTMAX <= 2 ? 4 : 3) * (W_BYTES + T * XROW);
    static constexpr int out_off = ring_bytes;
    static constexpr int bar_off = out_off + T * OUT_STRIDE * 4;
    static constexpr int misc_off = bar_off + (2 * MAX_STAGES + 8) * 8;   // full[], empty[], csync, fix done, fix request[5]
    // abort flag + stage geometry (32 B), deferred-reduction records (4 x 32 B), expert offsets, per-expert tile ranges
    static constexpr int pend_off = misc_off + 32;
    static constexpr int off_off = pend_off + 4 * 32;
    static constexpr int rng_off = off_off + (MOQE_MAX_EXPERTS + 2) * 4;
    static constexpr int total = rng_off + 2 * MOQE_MAX_EXPERTS * 4;
    static constexpr int dyn_bytes = total + 128;
};

// static work decomposition (see "stream-K" below)
struct Sched {
    long long C;            // total cost
    int G, E, KB, TT;       // CTAs, experts, k-blocks per segment, tiles per expert (= ntiles*KB)
    int w[MOQE_MAX_EXPERTS];
    int split;
};

struct StreamParams {
    ExpertDev ex[MOQE_MAX_EXPERTS];
    Sched sched;
    const uint16_t* X;
    uint16_t* Y;
    const int32_t* perm;
    const int32_t* offsets;
    float* partials;        // [CTA][slot 0/1][chunk][T][128]
    uint32_t* counters;     // [expert][ntiles][chunk], zero on entry, left zero
    int* status;
    int M, N, K, Np, KB, E, ntiles;
};

__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// The packed words of chunk G (8 consecutive k) of the lane's two channel rows gl (lo) and gl + 8 (hi),
// gl = lane / 4, k quarter q = lane % 4, slot = q*8 + (gl ^ 2q), read from the warp's blob in shared
// memory.  4-bit: one word per row; 8-bit: two words per row; 3-bit pieces are three words that serve
// all four chunks, so they are fetched once (G == 0) and kept.
template <int BITS>
struct LaneBlob { uint32_t lo[PieceWords<BITS>::n], hi[PieceWords<BITS>::n]; };

template <int BITS, int G>
__device__ __forceinline__ void load_chunk_smem(LaneBlob<BITS>& b, const unsigned char* blob, int slot) {
    if constexpr (BITS == 4) {
        b.lo[G] = *reinterpret_cast<const uint32_t*>(blob + slot * 16 + 4 * G);
        b.hi[G] = *reinterpret_cast<const uint32_t*>(blob + 512 + slot * 16 + 4 * G);
    } else if constexpr (BITS == 2) {
        if constexpr (G == 0) {          // one 16-byte slot holds the pieces of both rows
            const uint4 x = *reinterpret_cast<const uint4*>(blob + slot * 16);
            b.lo[0] = x.x; b.lo[1] = x.y;
            b.hi[0] = x.z; b.hi[1] = x.w;
        }
    } else if constexpr (BITS == 8) {
        const uint2 l = *reinterpret_cast<const uint2*>(blob + (G >> 1) * 512 + slot * 16 + 8 * (G & 1));
        const uint2 h = *reinterpret_cast<const uint2*>(blob + 1024 + (G >> 1) * 512 + slot * 16 + 8 * (G & 1));
        b.lo[2 * G] = l.x; b.lo[2 * G + 1] = l.y;
        b.hi[2 * G] = h.x; b.hi[2 * G + 1] = h.y;
    } else {
        if constexpr (G == 0) {
            const uint4 x = *reinterpret_cast<const uint4*>(blob + slot * 16);
            const uint2 y = *reinterpret_cast<const uint2*>(blob + 512 + slot * 8);
            b.lo[0] = x.x; b.lo[1] = x.y; b.lo[2] = x.z;
            b.hi[0] = x.w; b.hi[1] = y.x; b.hi[2] = y.y;
        }
    }
}

// ---------------------------------------------------------------------------
// Work decomposition ("stream-K" over packed tiles).
// All tiles of the call are laid out in one sequence [expert][channel tile nt][k-block kb]; tile
// (e, nt, kb) costs w[e] (about its bytes).  CTA c of G owns the tiles whose start cost lies in
// [c*C/G, (c+1)*C/G): a contiguous run, so every CTA carries the same cost to within one tile and
// has at most TWO partial pieces (its first and its last segment); everything between is whole
// (expert, nt) segments that need no reduction.  The decomposition is static (it does not depend
// on the routing), so an expert that received no rows simply leaves its CTAs idle.
// split == 0: whole segments are dealt round-robin instead (large batches: no partial sums).
// ---------------------------------------------------------------------------
struct Piece { int e, nt, kb0, kb1; };


__device__ __forceinline__ long long sched_base(const Sched& s, int e) {
    long long b = 0;
    for (int i = 0; i < e; ++i) b += (long long)s.TT * s.w[i];
    return b;
}
// first tile of expert e owned by CTA c or a later CTA
__device__ __forceinline__ int sched_tbegin(const Sched& s, int c, int e, long long base) {
    const long long num = (long long)c * s.C - base * s.G;
    if (num <= 0) return 0;
    const long long den = (long long)s.w[e] * s.G;
    const long long t = (num + den - 1) / den;
    return t > s.TT ? s.TT : (int)t;
}
__device__ __forceinline__ int sched_owner(const Sched& s, int e, long long base, int t) {
    return (int)(((base + (long long)t * s.w[e]) * s.G) / s.C);
}

// Walks the pieces of one CTA.  rng[2e], rng[2e+1] = the CTA's tile range inside expert e (split mode),
// computed once per CTA by sched_tbegin and kept in shared memory, so that next() needs no division by
// 64-bit numbers on the critical path.
struct PieceIter {
    int e, tb, te, seg;
    __device__ __forceinline__ void init(int cta) { e = -1; tb = te = 0; seg = cta; }
    __device__ __forceinline__ bool next(const Sched& s, int ntiles, const volatile int* rng, Piece& pc) {
        if (!s.split) {                                   // whole segments, round-robin
            if (seg >= s.E * ntiles) return false;
            pc.e = seg / ntiles;
            pc.nt = seg - pc.e * ntiles;
            pc.kb0 = 0;
            pc.kb1 = s.KB;
            seg += s.G;
            return true;
        }
        for (;;) {
            if (e >= 0 && tb < te) {
                const int sg = tb / s.KB;
                pc.e = e;
                pc.nt = sg;
                pc.kb0 = tb - sg * s.KB;
                const int len = min(s.KB - pc.kb0, te - tb);
                pc.kb1 = pc.kb0 + len;
                tb += len;
                return true;
            }
            if (++e >= s.E) return false;
            tb = rng[2 * e];
            te = rng[2 * e + 1];
        }
    }
};

constexpr int MAX_CHUNKS_SPLIT = 2;          // split mode is used for M <= 64 rows: at most two 32-row chunks per expert
constexpr int MAX_PENDING = 2 * MAX_CHUNKS_SPLIT;

// consumer-wide barrier (8 warps) on an mbarrier so that the wait is bounded like every other
struct ConsumerSync {
    uint32_t bar, phase;
    __device__ __forceinline__ bool sync(volatile int* abort_flag, int* status) {
        __syncwarp();
        if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
        const bool ok = __all_sync(0xffffffffu, mbar_wait(bar, phase, abort_flag, status));   // warp-uniform verdict
        phase ^= 1u;
        return ok;
    }
};

// Independent partial-sum sets per thread: consecutive MMAs go to different sets so that they do not wait
// for one another (a dependent mma.sync chain would make every tile cost its full pipeline latency).
template <int NT> struct Sets { static constexpr int n = NT <= 2 ? 2 : 1; };

// acc += scale * (sum of sets FIRST .. FIRST+COUNT-1  -  zf * xs), then clear those sets and xs.
// XS: the sets hold sum X*(128+c) and xs holds sum X (from the all-ones MMA); zf = 128 + zero-point.
template <int NT, int FIRST, int COUNT, int NSETS, bool XS>
__device__ __forceinline__ void promote_sets(float (&acc)[NT][4], float (&part)[NSETS][NT][4], float (&xs)[NT][4], float sl,
                                             float sh, float zfl, float zfh) {
#pragma unroll
    for (int t = 0; t < NT; ++t) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float v = part[FIRST][t][j];
#pragma unroll
            for (int c = 1; c < COUNT; ++c) v += part[FIRST + c][t][j];
            if constexpr (XS) {
                v = fmaf(-(j < 2 ? zfl : zfh), xs[t][j], v);
                xs[t][j] = 0.f;
            }
            acc[t][j] = fmaf(j < 2 ? sl : sh, v, acc[t][j]);
#pragma unroll
            for (int c = 0; c < COUNT; ++c) part[FIRST + c][t][j] = 0.f;
        }
    }
}

// One k-block (one ring stage) for one consumer warp: NT column blocks of 8 tokens.
// 4- and 3-bit codes enter the MMA as 128 + c (two instructions per pair of codes); a second MMA per k-step
// against an all-ones operand yields sum_k X, and (128 + z) * sum_k X is removed when the group is promoted.
// 8-bit codes enter as c - z directly.  pc_zl / pc_zh: zero-points of the lane's two channel rows when the
// expert is per-channel (or symmetric).
// GM: groups per tile (0 = per-channel expert, 1, 2 or 4) -- a template parameter, like every other switch in
// here, so that the whole k-block is ONE basic block and the four chunks overlap in the instruction stream.
template <int BITS, int NT, int NSETS, int GM>
__device__ __forceinline__ void consume_stage(const unsigned char* stage, int x_off, int warp, int gl, int q,
                                              bool has_zeros, float pc_zl, float pc_zh, float (&acc)[NT][4],
                                              float (&part)[NSETS][NT][4], float (&xs)[NT][4]) {
    constexpr bool XS = BITS != 8;
    const int slot = q * 8 + (gl ^ (2 * q));
    LaneBlob<BITS> b;
    const unsigned char* blob = stage + warp * moqe_blob_bytes(BITS);
    constexpr bool per_channel = GM == 0;
    constexpr int ngrp = GM == 0 ? 1 : GM;
    const int hz = has_zeros ? 1 : 0, row = warp * 16 + gl;
    const unsigned char* xrow = stage + x_off + gl * XROW + 16 * q;
    // scale / zero-point of the current group for the lane's two channel rows (reloaded where a group begins)
    float zlg = pc_zl, zhg = pc_zh, slg = 0.f, shg = 0.f;
    constexpr uint32_t ONES = 0x3F803F80u;
    auto chunk = [&](auto Gc) {
        constexpr int G = decltype(Gc)::value;
        constexpr int S = G % NSETS;
        constexpr int gj = ngrp == 4 ? G : (ngrp == 2 ? (G >> 1) : 0);
        constexpr bool group_begins = ngrp == 4 || (ngrp == 2 && (G & 1) == 0) || G == 0;
        if constexpr (!per_channel && group_begins) {
            const __half* sc = moqe_tile_scales(stage, BITS, hz, gj) + row;
            slg = __half2float(sc[0]) * (BITS == 8 ? W8_PRESCALE : 1.f);
            shg = __half2float(sc[8]) * (BITS == 8 ? W8_PRESCALE : 1.f);
            // symmetric experts have no zero-point rows: the (in-bounds) loads below are then ignored
            const __nv_bfloat16* zp = moqe_tile_zeros(stage, BITS, gj) + row;
            const float zl_t = __bfloat162float(zp[0]), zh_t = __bfloat162float(zp[8]);
            zlg = has_zeros ? zl_t : pc_zl;
            zhg = has_zeros ? zh_t : pc_zh;
        }
        load_chunk_smem<BITS, G>(b, blob, slot);
        uint32_t lo[4], hi[4];
        if constexpr (XS) {
            unpack_chunk_biased<BITS, G>(b.lo, lo);
            unpack_chunk_biased<BITS, G>(b.hi, hi);
        } else {
            unpack_chunk<BITS, G>(b.lo, zlg, lo);
            unpack_chunk<BITS, G>(b.hi, zhg, hi);
        }
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            const uint4 xb = *reinterpret_cast<const uint4*>(xrow + t * 8 * XROW + G * 64);   // 8 tokens x this chunk's k
            mma_bf16(part[S][t], lo[0], hi[0], lo[1], hi[1], xb.x, xb.y);
            mma_bf16(part[S][t], lo[2], hi[2], lo[3], hi[3], xb.z, xb.w);
            if constexpr (XS) {
                mma_bf16(xs[t], ONES, ONES, ONES, ONES, xb.x, xb.y);
                mma_bf16(xs[t], ONES, ONES, ONES, ONES, xb.z, xb.w);
            }
        }
        if constexpr (!per_channel) {
            const float zfl = 128.f + zlg, zfh = 128.f + zhg;
            if constexpr (ngrp == 4) {
                promote_sets<NT, S, 1, NSETS, XS>(acc, part, xs, slg, shg, zfl, zfh);
            } else if constexpr (ngrp == 2) {
                if constexpr ((G & 1) == 1) {
                    if constexpr (NSETS == 4) promote_sets<NT, G - 1, 2, NSETS, XS>(acc, part, xs, slg, shg, zfl, zfh);
                    else promote_sets<NT, 0, NSETS, NSETS, XS>(acc, part, xs, slg, shg, zfl, zfh);
                }
            } else {
                if constexpr (G == 3) promote_sets<NT, 0, NSETS, NSETS, XS>(acc, part, xs, slg, shg, zfl, zfh);
            }
        }
    };
    chunk(std::integral_constant<int, 0>{});
    chunk(std::integral_constant<int, 1>{});
    chunk(std::integral_constant<int, 2>{});
    chunk(std::integral_constant<int, 3>{});
}

// The k-block loop of one (piece, token chunk) for one consumer warp, specialised on the code width and the
// number of 8-token column blocks; leaves the warp's [tokens][16 channels] fp32 results in the CTA's staging
// tile `out`.  Deliberately NOT inlined: as a function of its own it gets the whole register budget for its
// accumulators, instead of sharing it with everything the scheduling code around it keeps alive.
// state: ring stage (bits 0-7), ring phase (bit 8), consumer-barrier phase (bit 9); returns the new state,
// or -1 if a wait was abandoned.
template <int BITS, int NT, int GM>
__device__ __noinline__ int mainloop_to_out(const StreamParams* pp, int e, int nt, int kb0, int kb1, int state, int nstg,
                                            int stage_bytes, int x_off,
                                            const unsigned char* smem, uint32_t bar_full, uint32_t bar_empty, uint32_t bar_csync,
                                            volatile int* s_abort, float* out) {
    constexpr int NSETS = Sets<NT>::n;
    const StreamParams& p = *pp;
    const ExpertDev& ex = p.ex[e];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gl = lane >> 2, q = lane & 3;
    Ring ring;
    ring.stage = state & 0xFF;
    ring.phase = (state >> 8) & 1;
    ConsumerSync cs{bar_csync, (uint32_t)((state >> 9) & 1)};
    const bool has_zeros = ex.has_zeros != 0;
    const int n_lo = nt * 128 + warp * 16 + gl;                          // this lane's channel rows: n_lo, n_lo + 8
    float s_lo = 0.f, s_hi = 0.f;                                         // per-channel scales and zero-points
    float pc_zl = (float)(1 << (BITS - 1)), pc_zh = pc_zl;
    if constexpr (GM == 0) {
        s_lo = __half2float(ex.scales_pc[n_lo]) * (BITS == 8 ? W8_PRESCALE : 1.f);
        s_hi = __half2float(ex.scales_pc[n_lo + 8]) * (BITS == 8 ? W8_PRESCALE : 1.f);
        if (has_zeros) { pc_zl = __bfloat162float(ex.zeros_pc[n_lo]); pc_zh = __bfloat162float(ex.zeros_pc[n_lo + 8]); }
    }
    float acc[NT][4], part[NSETS][NT][4], xs[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            acc[i][j] = xs[i][j] = 0.f;
#pragma unroll
            for (int c = 0; c < NSETS; ++c) part[c][i][j] = 0.f;
        }
#pragma unroll 1
    for (int kb = kb0; kb < kb1; ++kb) {
        if (!__all_sync(0xffffffffu, mbar_wait(bar_full + 8 * ring.stage, ring.phase, s_abort, p.status))) return -1;
        consume_stage<BITS, NT, NSETS, GM>(smem + ring.stage * stage_bytes, x_off, warp, gl, q, has_zeros, pc_zl, pc_zh, acc,
                                       part, xs);
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty + 8 * ring.stage);
        ring.advance(nstg);
    }
    if constexpr (GM == 0) {
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float v = part[0][t][j];
#pragma unroll
                for (int c = 1; c < NSETS; ++c) v += part[c][t][j];
                if constexpr (BITS != 8) v = fmaf(-(128.f + (j < 2 ? pc_zl : pc_zh)), xs[t][j], v);
                acc[t][j] = (j < 2 ? s_lo : s_hi) * v;
            }
    }
    if (!cs.sync(s_abort, p.status)) return -1;                         // previous readers of `out` are done
#pragma unroll
    for (int t = 0; t < NT; ++t) {
        const int tok = t * 8 + 2 * q, nl = warp * 16 + gl;
        out[tok * OUT_STRIDE + nl] = acc[t][0];
        out[(tok + 1) * OUT_STRIDE + nl] = acc[t][1];
        out[tok * OUT_STRIDE + nl + 8] = acc[t][2];
        out[(tok + 1) * OUT_STRIDE + nl + 8] = acc[t][3];
    }
    if (!cs.sync(s_abort, p.status)) return -1;
    return ring.stage | (int)(ring.phase << 8) | (int)(cs.phase << 9);
}

template <int NTMAX>
__global__ void __launch_bounds__(STREAM_THREADS, 2) qgemm_stream_kernel(const __grid_constant__ StreamParams p) {
    using L = StreamSmem<NTMAX>;
    constexpr int T = L::T;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_full = sbase + L::bar_off, bar_empty = bar_full + 8 * MAX_STAGES, bar_csync = bar_empty + 8 * MAX_STAGES;
    const uint32_t bar_fixdone = bar_csync + 8, bar_fixreq = bar_csync + 16;   // bar_fixreq[k], k <= MAX_PENDING: one per request
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::misc_off);
    volatile int* s_geom = reinterpret_cast<volatile int*>(smem + L::misc_off + 16);   // {stages, stage bytes, x offset}
    volatile int* s_pend = reinterpret_cast<volatile int*>(smem + L::pend_off);        // [MAX_PENDING][8] deferred reductions
    volatile int* s_off = reinterpret_cast<volatile int*>(smem + L::off_off);          // expert row offsets
    volatile int* s_rng = reinterpret_cast<volatile int*>(smem + L::rng_off);          // this CTA's tile range per expert
    const Sched& sch = p.sched;

    // ---- prologue: needs nothing but the launch parameters, so under programmatic dependent launch it
    // ---- overlaps the tail of the previous kernel in the stream
    if (tid == 0) {
        for (int i = 0; i < MAX_STAGES; ++i) { mbar_init(bar_full + 8 * i, 33); mbar_init(bar_empty + 8 * i, CONSUMER_WARPS); }
        mbar_init(bar_csync, CONSUMER_WARPS);
        for (int i = 0; i <= MAX_PENDING; ++i) mbar_init(bar_fixreq + 8 * i, CONSUMER_WARPS);
        mbar_init(bar_fixdone, 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid >= 32 && tid < 32 + sch.E) {                    // this CTA's tile range inside each expert
        const int e = tid - 32;
        int tb = 0, te = 0;
        if (sch.split) {
            const long long base = sched_base(sch, e);
            tb = sched_tbegin(sch, blockIdx.x, e, base);
            te = sched_tbegin(sch, blockIdx.x + 1, e, base);
        }
        s_rng[2 * e] = tb;
        s_rng[2 * e + 1] = te;
    }
    __syncthreads();
    if (tid == 0) {
        // stage size: the largest packed tile among the experts this CTA's (static) share of the work touches
        int wmax = 0;
        for (int e = 0; e < sch.E; ++e)
            if (!sch.split || s_rng[2 * e] < s_rng[2 * e + 1]) wmax = max(wmax, p.ex[e].tile_stride);
        const int x_off = (wmax + 127) & ~127;
        const int stage_bytes = x_off + T * XROW;
        s_geom[0] = min(MAX_STAGES, L::ring_bytes / stage_bytes);
        s_geom[1] = stage_bytes;
        s_geom[2] = x_off;
    }
    // from here on the previous kernel's results are needed (sort tables, activations, workspace); the next
    // kernel may start its own prologue as soon as this one's CTAs make room
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid <= sch.E) s_off[tid] = p.offsets[tid];
    __syncthreads();
    const int nstg = s_geom[0], stage_bytes = s_geom[1], x_off = s_geom[2];

    if (warp == CONSUMER_WARPS) {
        // ------------------------------------------------------------------ producer warp
        Ring ring;
        bool ok = true;
        PieceIter it;
        it.init(blockIdx.x);
        Piece pc;
        while (ok && it.next(sch, p.ntiles, s_rng, pc)) {
            const int row0 = s_off[pc.e], rows = s_off[pc.e + 1] - row0;
            if (rows <= 0) continue;
            const ExpertDev& ex = p.ex[pc.e];
            const uint32_t wbytes = (uint32_t)ex.tile_stride;                     // codes + the tile's scales / zero-points
            const uint8_t* wsrc = ex.tiles + (size_t)pc.nt * p.KB * wbytes;
            for (int c0 = 0; ok && c0 < rows; c0 += T) {
                const int tvalid = min(T, rows - c0);
                const int my_row = lane < tvalid ? p.perm[row0 + c0 + lane] : 0;
                for (int kb = pc.kb0; kb < pc.kb1; ++kb) {
                    if (!(ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * ring.stage, ring.phase ^ 1u, s_abort, p.status)))) break;
                    const uint32_t stage = sbase + ring.stage * stage_bytes;
                    const uint32_t full = bar_full + 8 * ring.stage;
                    if (lane == 0) {                                              // one bulk copy: the packed tile
                        mbar_expect_tx(full, wbytes);
                        bulk_load(stage, wsrc + (size_t)kb * wbytes, wbytes, full);
                    }
                    // the expert's token rows for these 128 k, gathered through perm with 16-byte async copies
                    // (zero-filled beyond K); each lane's copies report to the stage's barrier when they land
                    for (int id0 = 0; id0 < tvalid * 16; id0 += 32) {            // tvalid*16 is a multiple of 16: whole or half warps
                        const int id = id0 + lane;
                        const int r = id >> 4, c16 = id & 15;
                        const int src_row = __shfl_sync(0xffffffffu, my_row, r & 31);
                        if (id >= tvalid * 16) continue;
                        const int k = kb * 128 + c16 * 8;
                        const int nbytes = max(0, min(16, (p.K - k) * 2));
                        const uint16_t* src = nbytes > 0 ? p.X + (size_t)src_row * p.K + k : p.X;
                        cp_async16(stage + x_off + r * XROW + c16 * 16, src, nbytes);
                    }
                    cp_async_arrive_noinc(full);
                    ring.advance(nstg);
                }
            }
        }
    } else if (warp == CONSUMER_WARPS + 1) {
        // ------------------------------------------------------------------ fix-up warp
        // Announces this CTA's partial sums to the rest of the grid -- a fence and an atomic, two round trips to
        // L2 -- so that the consumer warps never wait for them.  Request k is record k of s_pend, filled in by
        // consumer thread 0 before the consumers arrive on bar_fixreq; rec[0] < 0 is the closing request.
        if (lane == 0) {
            for (int k = 0; k <= MAX_PENDING; ++k) {
                if (!mbar_wait(bar_fixreq + 8 * k, 0, s_abort, p.status)) break;
                volatile int* rec = s_pend + 8 * (k < MAX_PENDING ? k : 0);
                if (k >= MAX_PENDING || rec[0] < 0) break;
                const int e = rec[1], nt = rec[2], chunk = rec[5];
                const long long base = sched_base(sch, e);
                const int c_first = sched_owner(sch, e, base, nt * p.KB);
                const int c_last = sched_owner(sch, e, base, nt * p.KB + p.KB - 1);
                unsigned* cnt = p.counters + ((size_t)e * p.ntiles + nt) * MAX_CHUNKS_SPLIT + chunk;
                __threadfence();                                   // the consumers' partial stores, observed through the barrier
                const unsigned old = atomicAdd(cnt, 1u);
                const int last = (old == (unsigned)(c_last - c_first));
                if (last) *cnt = 0u;                               // leave the counters clear for the next call
                int slots = 0;                                     // bit i: contributor c_first + i parked its piece in slot 1
                if (last)
                    for (int cc = c_first; cc <= c_last && cc - c_first < 24; ++cc)
                        if (sched_tbegin(sch, cc, e, base) <= nt * p.KB) slots |= 1 << (cc - c_first);
                rec[6] = c_first;
                rec[7] = (c_last - c_first) | (slots << 8);
                rec[0] = last;
            }
            mbar_arrive(bar_fixdone);
        }
    } else {
        // ------------------------------------------------------------------ consumer warps
        float* out = reinterpret_cast<float*>(smem + L::out_off);
        Ring ring;
        ConsumerSync cs{bar_csync, 0};
        bool ok = true;
        int n_pending = 0;                                   // partial pieces handed to the fix-up warp
        PieceIter it;
        it.init(blockIdx.x);
        Piece pc;
        while (ok && it.next(sch, p.ntiles, s_rng, pc)) {
            const int row0 = s_off[pc.e], rows = s_off[pc.e + 1] - row0;
            if (rows <= 0) continue;
            const ExpertDev& ex = p.ex[pc.e];
            const bool whole = pc.kb0 == 0 && pc.kb1 == p.KB;
            for (int c0 = 0, chunk = 0; ok && c0 < rows; c0 += T, ++chunk) {
                const int tvalid = min(T, rows - c0);
                const int nt_run = tvalid <= 8 ? 1 : (tvalid <= 16 ? 2 : 4);
                const int state = ring.stage | (int)(ring.phase << 8) | (int)(cs.phase << 9);
                const int gm = moqe_groups_per_tile(ex.group);
                int ns;
#define MOQE_MAIN_ARGS (&p, pc.e, pc.nt, pc.kb0, pc.kb1, state, nstg, stage_bytes, x_off, smem, bar_full, bar_empty, bar_csync, s_abort, out)
#define MOQE_MAIN(B, NTV)                                                                                   \
    (gm == 0 ? mainloop_to_out<B, NTV, 0> MOQE_MAIN_ARGS : gm == 1 ? mainloop_to_out<B, NTV, 1> MOQE_MAIN_ARGS  \
     : gm == 2 ? mainloop_to_out<B, NTV, 2> MOQE_MAIN_ARGS : mainloop_to_out<B, NTV, 4> MOQE_MAIN_ARGS)
#define MOQE_MAIN_NT(B)                                                                          \
    do {                                                                                         \
        if (NTMAX == 1 || nt_run == 1) ns = MOQE_MAIN(B, 1);                                     \
        else if (NTMAX == 2 || nt_run == 2) ns = MOQE_MAIN(B, (NTMAX >= 2 ? 2 : 1));             \
        else ns = MOQE_MAIN(B, (NTMAX >= 4 ? 4 : 1));                                            \
    } while (0)
                if (ex.bits == 4) MOQE_MAIN_NT(4);
                else if (ex.bits == 8) MOQE_MAIN_NT(8);
                else if (ex.bits == 2) MOQE_MAIN_NT(2);
                else MOQE_MAIN_NT(3);
#undef MOQE_MAIN_NT
#undef MOQE_MAIN
#undef MOQE_MAIN_ARGS
                if (ns < 0) { ok = false; break; }
                ring.stage = ns & 0xFF;
                ring.phase = (uint32_t)(ns >> 8) & 1u;
                cs.phase = (uint32_t)(ns >> 9) & 1u;
                // `out` now holds this chunk's [tokens][128 channels] fp32 tile (all warps have written and synchronised)
                const int j0 = row0 + c0;
                if (whole) {
                    // the whole K of this segment was ours: round and store rows at their original positions
                    for (int i = tid; i < tvalid * 64; i += CONSUMER_WARPS * 32) {
                        const int tok = i >> 6, v = i & 63;
                        const int n = pc.nt * 128 + v * 2;
                        if (n >= p.N) continue;                                 // N is even
                        const int dst = p.perm[j0 + tok];
                        *reinterpret_cast<uint32_t*>(p.Y + (size_t)dst * p.N + n) =
                            pack_bf16x2(out[tok * OUT_STRIDE + v * 2], out[tok * OUT_STRIDE + v * 2 + 1]);
                    }
                } else {
                    // partial sum: park it in this CTA's slot and hand the announcement to the fix-up warp; whichever
                    // CTA announces last for the segment adds the slots up after finishing its own work
                    const int slot = pc.kb0 != 0 ? 0 : 1;
                    float* dst = p.partials + (((size_t)blockIdx.x * 2 + slot) * MAX_CHUNKS_SPLIT + chunk) * (T * 128);
                    for (int i = tid; i < tvalid * 32; i += CONSUMER_WARPS * 32) {
                        const int tok = i >> 5, v = i & 31;
                        *reinterpret_cast<float4*>(dst + tok * 128 + v * 4) = *reinterpret_cast<const float4*>(out + tok * OUT_STRIDE + v * 4);
                    }
                    if (tid == 0 && n_pending < MAX_PENDING) {
                        volatile int* rec = s_pend + 8 * n_pending;
                        rec[0] = 0; rec[1] = pc.e; rec[2] = pc.nt; rec[3] = j0; rec[4] = tvalid; rec[5] = chunk;
                    }
                    __syncwarp();
                    if (lane == 0 && n_pending < MAX_PENDING) mbar_arrive(bar_fixreq + 8 * n_pending);   // releases this warp's stores and the record
                    ++n_pending;
                }
            }
        }
        // ---- close the fix-up warp's queue, then add up the segments this CTA was the last to announce --------
        if (tid == 0 && n_pending < MAX_PENDING) s_pend[8 * n_pending] = -1;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_fixreq + 8 * min(n_pending, MAX_PENDING));
        if (ok && n_pending > 0 && __all_sync(0xffffffffu, mbar_wait(bar_fixdone, 0, s_abort, p.status))) {
            for (int pi = 0; pi < n_pending && pi < MAX_PENDING; ++pi) {
                volatile int* rec = s_pend + 8 * pi;
                if (rec[0] != 1) continue;                   // the fix-up warp's atomic and the barrier order the reads below
                const int nt = rec[2], pend_j0 = rec[3], pend_tv = rec[4], pend_chunk = rec[5];
                const int c_first = rec[6], n_contrib = (rec[7] & 0xFF) + 1, slots = rec[7] >> 8;
                for (int i = tid; i < pend_tv * 64; i += CONSUMER_WARPS * 32) {
                    const int tok = i >> 6, v = i & 63;
                    const int n = nt * 128 + v * 2;
                    if (n >= p.N) continue;
                    float a = 0.f, b = 0.f;
                    for (int ci = 0; ci < n_contrib; ++ci) {
                        // a contributor whose piece starts at the segment's start parked it in slot 1, else in slot 0
                        const int slot = (slots >> ci) & 1;
                        const float* src = p.partials + (((size_t)(c_first + ci) * 2 + slot) * MAX_CHUNKS_SPLIT + pend_chunk) * (T * 128);
                        const float2 pv = __ldcg(reinterpret_cast<const float2*>(src + tok * 128 + v * 2));
                        a += pv.x;
                        b += pv.y;
                    }
                    const int dst = p.perm[pend_j0 + tok];
                    *reinterpret_cast<uint32_t*>(p.Y + (size_t)dst * p.N + n) = pack_bf16x2(a, b);
                }
            }
        }
    }
    __syncthreads();
    if (*s_abort) {
        // let bulk copies that may still be in flight land before the shared memory is released
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
    }
}

int pick_ntmax(int M) { return M <= 8 ? 1 : (M <= 16 ? 2 : 4); }

constexpr int MAX_GRID = 512;                 // bound on resident CTAs the partial slots are sized for

int sm_count() {                              // of the current device (asked every time: a process may drive several)
    int dev = 0, n = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n > 0 ? n : 148;
}

// relative cost of one packed tile in the work split.  Measured: a tile costs about the same time whatever its
// width (the per-tile latency of a consumer warp, not its bytes, sets the pace), hence equal costs.
int g_tile_cost[9] = {0, 0, 8, 8, 8, 0, 0, 0, 8};

}  // namespace

void stream_set_tile_cost(int bits, int cost) { if (bits >= 0 && bits <= 8 && cost > 0) g_tile_cost[bits] = cost; }

size_t stream_zero_bytes(int M, int Np) {
    if (M > SPLIT_MAX_ROWS) return 0;
    return (size_t)MOQE_MAX_EXPERTS * (Np / 128) * MAX_CHUNKS_SPLIT * sizeof(uint32_t);
}

size_t stream_workspace_bytes(int M, int Np, int E) {
    (void)E;
    if (M > SPLIT_MAX_ROWS) return 0;
    size_t counters = (stream_zero_bytes(M, Np) + 255) / 256 * 256;
    size_t partials = (size_t)MAX_GRID * 2 * MAX_CHUNKS_SPLIT * (8 * pick_ntmax(M)) * 128 * sizeof(float);
    return counters + partials;
}

moqe_status launch_qgemm_stream(const void* X, int M, int N, int K, const moqe_expert* const* ex, int E, void* Y,
                                const int32_t* perm, const int32_t* offsets, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (M == 0) return MOQE_OK;
    StreamParams p;
    p.KB = ex[0]->Kp / 128;
    p.Np = ex[0]->Np;
    p.ntiles = p.Np / 128;
    Sched& s = p.sched;
    s.E = E;
    s.KB = p.KB;
    s.TT = p.ntiles * p.KB;
    s.C = 0;
    for (int e = 0; e < E; ++e) {
        p.ex[e] = ex[e]->dev();
        s.w[e] = g_tile_cost[ex[e]->bits];
        s.C += (long long)s.TT * s.w[e];
    }
    s.split = M <= SPLIT_MAX_ROWS ? 1 : 0;
    int ctas = 2 * sm_count();
    if (ctas > MAX_GRID) ctas = MAX_GRID;
    // split mode: every CTA's cost share must be at least one tile of the dearest kind, so that every CTA
    // between the owners of a segment's first and last tile really owns a tile of it (the reduction counts them)
    int wmax = 1;
    for (int e = 0; e < E; ++e) wmax = s.w[e] > wmax ? s.w[e] : wmax;
    const long long work_items = s.split ? s.C / wmax : (long long)E * p.ntiles;
    long long grid_ll = work_items < ctas ? (work_items < 1 ? 1 : work_items) : ctas;
    if (s.split) {
        // the reduction records which slot each contributor used in a 24-bit mask: keep a segment's contributors
        // below that (one segment costs KB * w, one CTA carries C / G)
        const long long cap = 22 * s.C / ((long long)p.KB * wmax);
        if (grid_ll > cap) grid_ll = cap < 1 ? 1 : cap;
    }
    const int grid = (int)grid_ll;
    s.G = grid;
    p.X = (const uint16_t*)X;
    p.Y = (uint16_t*)Y;
    p.perm = perm;
    p.offsets = offsets;
    p.M = M; p.N = N; p.K = K; p.E = E;
    p.status = device_status_word();
    p.counters = nullptr;
    p.partials = nullptr;
    if (s.split) {
        if (!ws || ws_bytes < stream_workspace_bytes(M, p.Np, E)) return MOQE_ERR_WORKSPACE;
        p.counters = (uint32_t*)ws;
        p.partials = (float*)((char*)ws + (stream_zero_bytes(M, p.Np) + 255) / 256 * 256);
    }
    const int nt = pick_ntmax(M);
    cudaError_t err = cudaSuccess;
#define MOQE_LAUNCH(NT)                                                                                           \
    do {                                                                                                          \
        const int smem = StreamSmem<NT>::dyn_bytes;                                                               \
        err = cudaFuncSetAttribute(qgemm_stream_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);   \
        if (err == cudaSuccess) {                                                                                 \
            cudaLaunchConfig_t cfg = {};                                                                          \
            cfg.gridDim = dim3(grid); cfg.blockDim = dim3(STREAM_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st; \
            cudaLaunchAttribute at[1];                                                                            \
            at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                        \
            at[0].val.programmaticStreamSerializationAllowed = 1;                                                 \
            cfg.attrs = at; cfg.numAttrs = 1;                                                                     \
            err = cudaLaunchKernelEx(&cfg, qgemm_stream_kernel<NT>, p);                                           \
        }                                                                                                         \
    } while (0)
    if (nt == 1) MOQE_LAUNCH(1);
    else if (nt == 2) MOQE_LAUNCH(2);
    else MOQE_LAUNCH(4);
#undef MOQE_LAUNCH
    if (err != cudaSuccess) return MOQE_ERR_CUDA;
    count_launch();
    return cuda_ok(cudaGetLastError());
}

}  // namespace moqe
