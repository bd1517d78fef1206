// Routed dequant-GEMM for decode shapes (at most 16 token rows in the batch): every touched
// expert's packed weights are streamed from HBM exactly once.
//
//   producer (1 thread)     : cp.async.bulk copies of whole packed 128x128-code tiles (codes + the
//                             tile's scales / zero-points, contiguous in HBM) into a shared-memory
//                             ring guarded by full/empty mbarriers.
//                             The copies carry an L2 evict-first policy: weights pass through L2 once.
//   dequant (4 warpgroups)  : warpgroup w takes the CTA's tiles t = w (mod 4).  Thread r of a
//                             warpgroup owns channel row r of the tile: it reads the row's packed
//                             words with conflict-free 128-bit shared loads, unpacks them in registers
//                             to the exact integers (c - z) in bf16 and stores them straight into
//                             TENSOR MEMORY (tcgen05.st, lane r) as operand A of the MMA -- no
//                             shared-memory round trip.  The same warpgroup fetches the token rows of
//                             its next tile (gathered through `perm`: the fused permutation) with
//                             16-byte async copies into a K-major, 128-byte-swizzled operand tile.
//                             Sixteen warps run this one loop, which is what hides the latency of the
//                             half-rate integer / bf16x2 instructions the unpacking consists of.
//   MMA issuer (1 warp)     : tcgen05.mma, A from TMEM (128 channels x 16 k), B = the token tile in
//                             shared memory (N = 16), fp32 accumulators in TMEM, one buffer per
//                             quantization group:
//                               Y[m][n] = sum_G s[n][G] * (sum_{k in G} X[m][k] * (c[n][k] - z[n][G]))
//                             so the tensor core only multiplies exactly representable numbers.
//                             The whole warp walks the tiles; one elected lane issues eight
//                             straight-line MMAs per tile and the commits.
//   epilogue (1 warpgroup)  : drains a finished group buffer (tcgen05.ld), multiplies by the group's
//                             fp32 scale, accumulates in registers, and at the end of a piece writes
//                             bf16 rows to their ORIGINAL positions (fused un-permutation) or parks an
//                             fp32 partial sum.
//
// Work split ("stream-K" over packed tiles): all tiles of the call form one sequence
// [expert][channel tile nt][k-block kb]; tile (e, nt, kb) costs w[e].  CTA c of G owns the tiles
// whose start cost lies in [c*C/G, (c+1)*C/G) -- equal work to within one tile, at most two partial
// pieces per CTA: a first one that starts inside its (expert, nt) segment and a last one that stops
// inside its segment.  A first piece is parked in the workspace and flagged as soon as it is done,
// early in the kernel; the CTA that holds the head of a segment -- its last piece -- keeps that sum in
// registers, adds the parked pieces of the following CTAs in CTA order (deterministic) and stores
// the rows.  All CTAs are resident (grid <= SM count), and the flag wait is bounded like every other.
//
// Takes experts that are per-channel or have groups of 128 k or more, and batches of at most 16
// rows; the caller routes everything else to the other kernels.
//
// Every mbarrier wait is bounded; on expiry the CTA raises its abort flag, latches
// MOQE_ERR_TIMEOUT, lets copies in flight land, frees its TMEM and returns.
//
// The operation is Section 3.1 of the paper (the selected quantization expert runs the sample);
// the paper describes no kernel.
#include <type_traits>

#include "dequant.cuh"
#include "tc_ptx.cuh"

namespace moqe {
namespace {

constexpr int TOK = 16;                                 // token columns of the MMA (rows of a batch)
constexpr int NWG = 4;                                  // dequant warpgroups; warpgroup w takes tiles t = w (mod 4)
constexpr int DQ_WARPS = 4 * NWG, MMA_WARP = DQ_WARPS, W_WARP = DQ_WARPS + 1;
constexpr int DEC_THREADS = (DQ_WARPS + 2) * 32;
constexpr int RING_BYTES = 134 * 1024;                  // packed-weight ring
constexpr int MAX_STAGES = 16;
constexpr int NA = 6;                                   // A-operand buffers in TMEM (64 columns each), tile t -> t % 6
constexpr int ND = 8;                                   // accumulator buffers (TOK columns each), group g -> g % 8
constexpr int NXS = 10;                                 // token-tile stages, tile t -> t % 10
constexpr int X_STAGE = TOK * 256;                      // TOK rows x 128 k bf16
constexpr int DONE_RING = 8;                            // "MMAs of tile t have completed" barriers, tile t -> t % 8
constexpr int TMEM_COLS = 512;
constexpr int D_COL0 = NA * 64;
static_assert(NA > NWG && ND >= 2 * NWG && D_COL0 + ND * TOK <= TMEM_COLS, "buffers: a warpgroup must not wait for the previous round");
constexpr int MAX_TILES = 512;                          // tiles one CTA can take (its tile table)

struct DecSmem {
    static constexpr int ring_off = 0;
    static constexpr int x_off = RING_BYTES;
    static constexpr int out_off = x_off + NXS * X_STAGE;             // float[NWG - 1][TOK][128]: a piece's shares
    static constexpr int bar_off = out_off + (NWG - 1) * TOK * 512;
    // wfull[16] wempty[16] afull[NA] done[8] turn[4] flush_free esync
    static constexpr int n_bars = 2 * MAX_STAGES + NA + DONE_RING + 4 + 1 + 1;
    static constexpr int misc_off = bar_off + n_bars * 8;              // tmem address, abort flag, ring geometry
    static constexpr int off_off = misc_off + 32;
    static constexpr int perm_off = off_off + (MOQE_MAX_EXPERTS + 2) * 4;   // perm of the batch's rows
    static constexpr int rng_off = perm_off + TOK * 4;
    static constexpr int ex_off = rng_off + 2 * MOQE_MAX_EXPERTS * 4;  // ExpertSm[MOQE_MAX_EXPERTS]
    static constexpr int tile_off = (ex_off + MOQE_MAX_EXPERTS * 64 + 15) & ~15;   // uint4[MAX_TILES]
    static constexpr int piece_off = tile_off + MAX_TILES * 16;        // int[MAX_TILES]: last tile of each piece
    static constexpr int total = piece_off + MAX_TILES * 4;
    static constexpr int dyn_bytes = total + 1024;                     // slack for manual 1024-byte alignment
};

// One call may carry several linear layers that share the routing (same rows, same perm): every (layer, expert)
// pair is one "expert" of the work split below, with its own packed tiles, shape, input and output.
struct DecSched {
    long long C;                    // total cost
    int G, E;                       // CTAs, (layer, expert) pairs
    int TT[MOQE_MAX_EXPERTS];       // tiles of the pair (= ntiles * KB of its layer)
    int w[MOQE_MAX_EXPERTS];        // cost of one of its tiles
};

struct DecParams {
    ExpertDev ex[MOQE_MAX_EXPERTS];
    DecSched sched;
    const uint16_t* X[MOQE_MAX_EXPERTS];    // per (layer, expert) pair: the layer's input, output and shape,
    uint16_t* Y[MOQE_MAX_EXPERTS];
    int N[MOQE_MAX_EXPERTS], K[MOQE_MAX_EXPERTS], KB[MOQE_MAX_EXPERTS];
    int rexp[MOQE_MAX_EXPERTS];             // and the routing expert whose rows it takes
    const int32_t* perm;
    const int32_t* offsets;
    float* partials;        // [CTA][TOK][128]: the partial sum of a CTA's first piece
    uint32_t* flags;        // [CTA]: that partial sum is parked; zero on entry, left zero
    int* status;
    int M, R;               // rows of the batch, routing experts
};

__device__ __forceinline__ long long dsched_base(const DecSched& s, int e) {
    long long b = 0;
    for (int i = 0; i < e; ++i) b += (long long)s.TT[i] * s.w[i];
    return b;
}
// first tile of expert e owned by CTA c or a later CTA
__device__ __forceinline__ int dsched_tbegin(const DecSched& s, int c, int e, long long base) {
    const long long num = (long long)c * s.C - base * s.G;
    if (num <= 0) return 0;
    const long long den = (long long)s.w[e] * s.G;
    const long long t = (num + den - 1) / den;
    return t > s.TT[e] ? s.TT[e] : (int)t;
}
__device__ __forceinline__ int dsched_owner(const DecSched& s, int e, long long base, int t) {
    return (int)(((base + (long long)t * s.w[e]) * s.G) / s.C);
}

// The CTA's tiles, in order, as a table in shared memory (one 16-byte entry per tile), built once by the whole CTA
// after the routing offsets are known: every role then reads its tile with one load instead of walking pieces.
//   x = kb | nt << 16        y = flags | e << 8 | rows << 16 | row0 << 24        z = accumulation-group index g
//   w = piece index | (the last CTA that owns a tile of this tile's (expert, nt) segment) << 16
// flags: first / last tile of its piece, ends / starts an accumulation group, piece = whole segment, piece starts
// inside its segment
// An accumulation group (one accumulator buffer handed to the epilogue) is: the whole piece for per-channel
// experts; for groups of 128 k or more, the k-blocks of one quantization group inside the piece (the scale is
// constant over the group, so a piece may cut it).
constexpr int TF_FIRST = 1, TF_LAST = 2, TF_ENDS = 4, TF_WHOLE = 8, TF_KB0NZ = 16, TF_GSTART = 32;

struct ExpertSm {            // per-expert facts of this CTA, in shared memory
    int tb, te;              // the CTA's tile range inside the expert ([nt][kb] order); empty if the expert has no rows
    int cum;                 // tiles of earlier experts
    int gbase;               // accumulation groups of earlier experts
    int gkb;                 // k-blocks per accumulation group (KB for per-channel experts)
    int row0, rows;
    int bits, group, has_zeros, stride;
    int pbase;               // pieces of earlier experts
    int KB, N, pad0, pad1;   // k-blocks per segment and output channels of its layer
};

struct Tile {
    int kb, nt, flags, e, rows, row0, g, piece, c_last;
    __device__ __forceinline__ explicit Tile(const uint4& v)
        : kb((int)(v.x & 0xFFFFu)), nt((int)(v.x >> 16)), flags((int)(v.y & 0xFFu)), e((int)((v.y >> 8) & 0xFFu)),
          rows((int)((v.y >> 16) & 0xFFu)), row0((int)(v.y >> 24)), g((int)v.z), piece((int)(v.w & 0xFFFFu)), c_last((int)(v.w >> 16)) {}
    __device__ __forceinline__ bool ends() const { return flags & TF_ENDS; }
};

// ---------------------------------------------------------------------------- dequant role
// Chunk G (8 consecutive k) of a piece as four bf16x2 registers holding the exact integers c - z.  `zc` is the
// tile's zero-point constant, packed once per tile: bf16x2(128 + z) for 4- and 3-bit codes (0x4300 | c is the
// bf16 number 128 + c), bf16x2(-z * 2^-13) for 8-bit codes (a zero-extended byte is the bf16 number c * 2^-133;
// one FMA with 2^120 gives (c - z) * 2^-13, and the fp32 scale carries the 2^13).
template <int BITS, int G>
__device__ __forceinline__ void unpack_chunk_zc(const uint32_t (&w)[PieceWords<BITS>::n], uint32_t zc, uint32_t* out) {
    if constexpr (BITS == 4) {
        const uint32_t v = w[G];
#pragma unroll
        for (int i = 0; i < 4; ++i) out[i] = hsub2_bf16(((v >> (4 * i)) & 0x000F000Fu) | 0x43004300u, zc);
    } else if constexpr (BITS == 3) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int pr = 4 * G + i;                 // pair index inside the piece
            uint32_t v;
            if (pr < 15) v = (w[pr / 5] >> (3 * (pr % 5))) & 0x00070007u;
            else v = ((w[0] >> 15) & 0x00010001u) | ((w[1] >> 14) & 0x00020002u) | ((w[2] >> 13) & 0x00040004u);
            out[i] = hsub2_bf16(v | 0x43004300u, zc);
        }
    } else {
        const uint32_t k120 = 0x7B807B80u;           // 2^120 in both halves
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t pair = __byte_perm(w[2 * G + (i >> 1)], 0u, (i & 1) ? 0x4342u : 0x4140u);
            __nv_bfloat162 r = __hfma2(*reinterpret_cast<const __nv_bfloat162*>(&pair), *reinterpret_cast<const __nv_bfloat162*>(&k120),
                                       *reinterpret_cast<const __nv_bfloat162*>(&zc));
            out[i] = *reinterpret_cast<uint32_t*>(&r);
        }
    }
}

// One packed tile -> operand A in tensor memory, for the thread that owns channel row `row` (= its TMEM lane).
// MMA k index k' = 32q + 8G + t holds the code of real k = 32G + 8q + t (piece q, chunk G): a piece then fills 16
// consecutive TMEM columns with one store, and the token-tile loader applies the same permutation to its
// 16-byte chunks.
template <int BITS>
__device__ __forceinline__ void dequant_tile(const unsigned char* stage, int row, uint32_t zc, uint32_t a_taddr) {
    const unsigned char* blob = stage + (row >> 4) * moqe_blob_bytes(BITS);
    const int half = (row >> 3) & 1, r = row & 7;
#pragma unroll 1
    for (int q = 0; q < 4; ++q) {
        uint32_t w[PieceWords<BITS>::n];
        load_piece_smem<BITS>(blob, half, q * 8 + (r ^ (2 * q)), w);
        uint32_t o[16];
        unpack_chunk_zc<BITS, 0>(w, zc, o);
        unpack_chunk_zc<BITS, 1>(w, zc, o + 4);
        unpack_chunk_zc<BITS, 2>(w, zc, o + 8);
        unpack_chunk_zc<BITS, 3>(w, zc, o + 12);
        tmem_st16(a_taddr + 16 * q, o);
    }
}

// The token rows of one tile (expert rows [row0, row0 + rows) of the sorted batch, k-block kb) as a K-major,
// 128-byte-swizzled UMMA operand: two halves of 64 k', each TOK rows x 128 bytes; 16-byte chunk (G, q) of real k
// goes to chunk 4q + G of k'.  Issued by the 128 threads of one warpgroup (t = thread index in it); k >= K is
// zero-filled.  Rows beyond `rows` are left as they are: their columns of the accumulator are never read.
__device__ __forceinline__ void load_token_tile(const uint16_t* X, int K, const volatile int* s_perm, uint32_t xs, int row0, int rows,
                                                int kb, int t) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int id = t + 128 * i, m = id >> 4, a = id & 15;
        if (m < rows) {
            const int src_row = s_perm[row0 + m];
            const int k = kb * 128 + a * 8;
            const int nbytes = max(0, min(16, (K - k) * 2));
            const uint16_t* src = nbytes > 0 ? X + (size_t)src_row * K + k : X;
            const int ap = 4 * (a & 3) + (a >> 2);
            cp_async16(xs + (ap >> 3) * (TOK * 128) + m * 128 + (((ap & 7) ^ (m & 7)) << 4), src, nbytes);
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// ---------------------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(DEC_THREADS, 1) qgemm_decode_kernel(const __grid_constant__ DecParams p) {
    using L = DecSmem;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + L::bar_off;
    const uint32_t bar_wfull = bar0, bar_wempty = bar0 + 8 * MAX_STAGES, bar_afull = bar_wempty + 8 * MAX_STAGES;
    const uint32_t bar_done = bar_afull + 8 * NA, bar_turn = bar_done + 8 * DONE_RING;
    const uint32_t bar_flushfree = bar_turn + 8 * 4, bar_esync = bar_flushfree + 8;
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + L::misc_off);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::misc_off + 4);
    volatile int* s_geom = reinterpret_cast<volatile int*>(smem + L::misc_off + 8);    // {stages, stage bytes, tiles}
    volatile int* s_off = reinterpret_cast<volatile int*>(smem + L::off_off);
    volatile int* s_rng = reinterpret_cast<volatile int*>(smem + L::rng_off);
    volatile int* s_perm = reinterpret_cast<volatile int*>(smem + L::perm_off);
    ExpertSm* s_ex = reinterpret_cast<ExpertSm*>(smem + L::ex_off);
    const uint4* s_tile = reinterpret_cast<const uint4*>(smem + L::tile_off);
    float* s_out = reinterpret_cast<float*>(smem + L::out_off);
    volatile int* s_piece = reinterpret_cast<volatile int*>(smem + L::piece_off);
    const DecSched& sch = p.sched;
    // warp-uniform bounded wait: every lane polls, the warp agrees on the verdict
    auto wwait = [&](uint32_t bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait_short(bar, parity, s_abort, p.status));
    };
    // one arrival per warp, after all its lanes are done with what the barrier hands over
    auto warrive = [&](uint32_t bar) {
        __syncwarp();
        if (lane == 0) mbar_arrive(bar);
    };
    // done[t % 8] completes when the MMAs of the CTA's t-th tile have
    auto wait_done = [&](int t) -> bool {
        return t < 0 || wwait(bar_done + 8 * (t & (DONE_RING - 1)), (uint32_t)(t >> 3) & 1u);
    };

    // ---- prologue: launch parameters only, so it may overlap the tail of the previous kernel in the stream
    if (tid == 0) {
        for (int i = 0; i < MAX_STAGES; ++i) { mbar_init(bar_wfull + 8 * i, 1); mbar_init(bar_wempty + 8 * i, 4); }
        for (int i = 0; i < NA; ++i) mbar_init(bar_afull + 8 * i, 4);
        for (int i = 0; i < DONE_RING; ++i) mbar_init(bar_done + 8 * i, 1);
        mbar_init(bar_turn, DQ_WARPS);                  // every dequant warp, once per piece
        mbar_init(bar_flushfree, 4);
        mbar_init(bar_esync, 4);                         // the four warps of the finalizing warpgroup
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid >= 32 && tid < 32 + sch.E) {                    // this CTA's tile range inside each expert
        const int e = tid - 32;
        const long long base = dsched_base(sch, e);
        s_rng[2 * e] = dsched_tbegin(sch, blockIdx.x, e, base);
        s_rng[2 * e + 1] = dsched_tbegin(sch, blockIdx.x + 1, e, base);
    }
    if (warp == MMA_WARP) tmem_alloc(sbase + L::misc_off, TMEM_COLS);
    // from here on the previous kernel's results are needed (sort tables, activations, workspace)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid <= p.R) s_off[tid] = p.offsets[tid];
    if (tid >= 64 && tid < 64 + TOK) s_perm[tid - 64] = tid - 64 < p.M ? p.perm[tid - 64] : 0;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) {
        // Per-expert facts, the ring geometry (stage = the largest packed tile this CTA will see) and the tile count:
        // lane e works out expert e (E <= 32), the running totals come from a warp scan -- one thread doing all
        // experts in turn costs the better part of a microsecond at every launch.
        const int e = lane;
        ExpertSm x = {};
        int cnt = 0, ng = 0, np = 0, str = 0;
        if (e < sch.E) {
            x.row0 = s_off[p.rexp[e]];
            x.rows = min(s_off[p.rexp[e] + 1] - x.row0, TOK);
            x.KB = p.KB[e]; x.N = p.N[e];
            x.tb = s_rng[2 * e];
            x.te = x.rows > 0 ? s_rng[2 * e + 1] : x.tb;
            x.bits = p.ex[e].bits; x.group = p.ex[e].group; x.has_zeros = p.ex[e].has_zeros; x.stride = p.ex[e].tile_stride;
            x.gkb = x.group == 0 ? x.KB : x.group / 128;
            if (x.te > x.tb) {
                cnt = x.te - x.tb;
                ng = x.te / x.gkb - x.tb / x.gkb + (x.te % x.gkb != 0 ? 1 : 0);
                np = (x.te - 1) / x.KB - x.tb / x.KB + 1;
                str = x.stride;
            }
        }
        int c = cnt, g = ng, q = np, wmax = str;            // inclusive scans / maximum over the lanes
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int c2 = __shfl_up_sync(0xffffffffu, c, d), g2 = __shfl_up_sync(0xffffffffu, g, d),
                      q2 = __shfl_up_sync(0xffffffffu, q, d);
            if (lane >= d) { c += c2; g += g2; q += q2; }
            wmax = max(wmax, __shfl_xor_sync(0xffffffffu, wmax, d));
        }
        if (e < sch.E) {
            x.cum = c - cnt;
            x.gbase = g - ng;
            x.pbase = q - np;
            s_ex[e] = x;
        }
        if (lane == 31) {
            const int stage_bytes = (max(wmax, 128) + 127) & ~127;
            s_geom[0] = min(MAX_STAGES, RING_BYTES / stage_bytes);
            s_geom[1] = stage_bytes;
            s_geom[2] = min(c, MAX_TILES);
            s_geom[3] = q;
        }
    }
    __syncthreads();
    const uint32_t tmem_base = *s_tmem;
    const int nstg = s_geom[0], stage_bytes = s_geom[1], T = s_geom[2], NP = s_geom[3];
    for (int i = tid; i < T; i += DEC_THREADS) {            // the tile table, one thread per tile
        int e = 0;
        while (e + 1 < sch.E && s_ex[e + 1].cum <= i) ++e;
        while (s_ex[e].te <= s_ex[e].tb) ++e;               // (experts without tiles share their successor's cum)
        const ExpertSm x = s_ex[e];
        const int KB = x.KB;
        const int tile = x.tb + i - x.cum, nt = tile / KB, kb = tile - nt * KB;
        const int kb0 = max(x.tb - nt * KB, 0), kb1 = min(x.te - nt * KB, KB);
        const bool last = kb + 1 == kb1;
        int flags = (kb == kb0 ? TF_FIRST : 0) | (last ? TF_LAST : 0) | ((last || (kb + 1) % x.gkb == 0) ? TF_ENDS : 0) |
                    ((kb0 == 0 && kb1 == KB) ? TF_WHOLE : 0) | (kb0 != 0 ? TF_KB0NZ : 0) |
                    ((kb == kb0 || kb % x.gkb == 0) ? TF_GSTART : 0);
        const int piece = x.pbase + nt - x.tb / KB;
        uint4 v;
        v.x = (uint32_t)kb | ((uint32_t)nt << 16);
        v.y = (uint32_t)flags | ((uint32_t)e << 8) | ((uint32_t)x.rows << 16) | ((uint32_t)x.row0 << 24);
        v.z = (uint32_t)(x.gbase + tile / x.gkb - x.tb / x.gkb);
        // owner of the segment's last tile (needed where the head of a split segment ends)
        v.w = (uint32_t)piece |
              ((last && kb0 == 0 && kb1 != KB) ? (uint32_t)dsched_owner(sch, e, dsched_base(sch, e), nt * KB + KB - 1) << 16 : 0u);
        if (last) s_piece[piece] = i;
        *reinterpret_cast<uint4*>(smem + L::tile_off + 16 * i) = v;
    }
    __syncthreads();

    if (warp == W_WARP) {
        // ------------------------------------------------------------------ packed-weight producer
        if (lane == 0) {
            Ring ring;
            const uint64_t once = l2_policy_evict_first();   // weights cross L2 once per call
            for (int t = 0; t < T; ++t) {
                const Tile ti(s_tile[t]);
                const uint32_t wbytes = (uint32_t)s_ex[ti.e].stride;
                if (!mbar_wait(bar_wempty + 8 * ring.stage, ring.phase ^ 1u, s_abort, p.status)) break;
                const uint32_t full = bar_wfull + 8 * ring.stage;
                mbar_expect_tx(full, wbytes);
                bulk_load_once(sbase + L::ring_off + ring.stage * stage_bytes,
                               p.ex[ti.e].tiles + ((size_t)ti.nt * s_ex[ti.e].KB + ti.kb) * wbytes, wbytes, full, once);
                ring.advance(nstg);
            }
        }
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------------------------ MMA issuer
        // The whole warp walks the tiles (warp-uniform control flow); one elected lane issues.  No accumulator
        // hand-shake is needed: buffer g % 8 is drained by the warpgroup that unpacked the group's last tile j before
        // it hands over its tile j + 8, and the group that reuses the buffer starts at tile j + 8 or later.
        const uint32_t idesc = umma_idesc(TOK);
        int a = 0, xst = 0;
        uint32_t aphase = 0;
        for (int t = 0; t < T; ++t) {
            const Tile ti(s_tile[t]);
            if (!wwait(bar_afull + 8 * a, aphase)) break;
            tc_fence_after();
            const uint32_t xs = sbase + L::x_off + xst * X_STAGE;
            const uint32_t dt = tmem_base + D_COL0 + (ti.g & (ND - 1)) * TOK, a0 = tmem_base + a * 64;
            const uint64_t b0 = umma_desc_sw128(xs), b1 = umma_desc_sw128(xs + TOK * 128);
            const uint32_t acc0 = (ti.flags & TF_GSTART) ? 0u : 1u;
            if (elect_one()) {
                umma_bf16_ts(dt, a0, b0, idesc, acc0);
                umma_bf16_ts(dt, a0 + 8, b0 + 2, idesc, 1u);
                umma_bf16_ts(dt, a0 + 16, b0 + 4, idesc, 1u);
                umma_bf16_ts(dt, a0 + 24, b0 + 6, idesc, 1u);
                umma_bf16_ts(dt, a0 + 32, b1, idesc, 1u);
                umma_bf16_ts(dt, a0 + 40, b1 + 2, idesc, 1u);
                umma_bf16_ts(dt, a0 + 48, b1 + 4, idesc, 1u);
                umma_bf16_ts(dt, a0 + 56, b1 + 6, idesc, 1u);
                umma_commit(bar_done + 8 * (t & (DONE_RING - 1)));
            }
            __syncwarp();
            if (++a == NA) { a = 0; aphase ^= 1u; }
            if (++xst == NXS) xst = 0;
        }
    } else if (warp < DQ_WARPS) {
        // ------------------------------------------------------------------ dequant warpgroups
        const int wg = warp >> 2, row = (warp & 3) * 32 + lane, twg = tid & 127;
        const uint32_t lane_taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        auto x_load = [&](int t) {                   // token rows of tile t (an empty group past the end)
            if (t < T) {
                const Tile xi(s_tile[t]);
                load_token_tile(p.X[xi.e], p.K[xi.e], s_perm, sbase + L::x_off + (t % NXS) * X_STAGE, xi.row0, xi.rows, xi.kb, twg);
            } else {
                asm volatile("cp.async.commit_group;" ::: "memory");
            }
        };
        float acc[TOK];                              // this warpgroup's share of the current piece, channel `row`
#pragma unroll
        for (int i = 0; i < TOK; ++i) acc[i] = 0.f;
        int flushed = 0;                             // pieces this warpgroup has handed to the finalizer
        // Accumulation groups that ended with this warpgroup's last two tiles and are not drained yet.  A group is
        // drained TWO rounds after its last tile was handed over: one round later its MMAs may still be queued behind
        // the other warpgroups' tiles, and waiting for them would put the MMA round trip into every round.
        struct Rec { int t, g, piece; float s; };
        Rec r0{-1, 0, 0, 0.f}, r1{-1, 0, 0, 0.f};    // two rounds back, previous round
        int acc_piece = -1;                          // the piece `acc` belongs to
        int last_t = -1, ph0 = 0, ph1 = 0;                        // pieces of this warpgroup's tiles of two rounds / one round ago
        bool ok = true;
        // scale and add a finished group (the caller knows that its MMAs have completed)
        auto drain = [&](Rec& r) {
            if (r.t < 0) return;
            tc_fence_after();
            uint32_t v[16];
            tmem_ld16(lane_taddr + D_COL0 + (r.g & (ND - 1)) * TOK, v);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < TOK; ++i) acc[i] = fmaf(r.s, __uint_as_float(v[i]), acc[i]);
            tc_fence_before();
            acc_piece = r.piece;
            r.t = -1;
        };
        // The last warpgroup of the chain also finishes the piece: with the sum of all four shares in registers it
        // stores the rows at their original positions (fused un-permutation), parks the sum, or adds the parked sums
        // of other CTAs.
        uint32_t esync_phase = 0;
        const int et = twg;
        auto finalize = [&](int q, float (&acc)[TOK]) -> bool {
            const Tile ti(s_tile[s_piece[q]]);       // the piece's last tile carries its facts
            const int n = ti.nt * 128 + row, j0 = ti.row0, rows = ti.rows, N = s_ex[ti.e].N;
            uint16_t* Y = p.Y[ti.e];
            if (ti.flags & TF_WHOLE) {
                // the whole K of this segment was ours: round and store rows at their original positions
                if (n < N) {
#pragma unroll
                    for (int m = 0; m < TOK; ++m)
                        if (m < rows) Y[(size_t)s_perm[j0 + m] * N + n] = __bfloat16_as_ushort(__float2bfloat16_rn(acc[m]));
                }
            } else if (ti.flags & TF_KB0NZ) {
                // A piece that starts inside its segment -- always a CTA's FIRST piece: park the partial sum and raise
                // this CTA's flag.  Nobody waits here: the barrier puts the 128 threads' stores before thread 0's
                // release, which publishes them together with the flag.
                float* dst = p.partials + (size_t)blockIdx.x * TOK * 128 + row;
#pragma unroll
                for (int m = 0; m < TOK; ++m)
                    if (m < rows) dst[m * 128] = acc[m];
                warrive(bar_esync);
                if (!wwait(bar_esync, esync_phase)) return false;
                esync_phase ^= 1u;
                if (et == 0) st_release_gpu(p.flags + blockIdx.x, 1u);
            } else {
                // The head of a segment whose tail belongs to the following CTAs -- always a CTA's LAST piece, while
                // the later pieces are parked by CTAs blockIdx.x + 1 .. c_last (each as its first piece).  Every thread
                // waits for their flags itself (bounded; an acquire load, so its reads of the parked sums need no
                // further fence), adds the sums in CTA order (deterministic) and stores.
                const int n_others = ti.c_last - (int)blockIdx.x;
                for (int c0 = 0; c0 < n_others; ++c0) {
                    const unsigned* f = p.flags + blockIdx.x + 1 + c0;
                    unsigned long long t_start = 0;
                    for (unsigned it = 1; ld_acquire_gpu(f) == 0u; ++it) {
                        if ((it & 63u) == 0) {
                            if (*s_abort) break;
                            const unsigned long long now = global_ns();
                            if (t_start == 0) t_start = now;
                            else if (now - t_start > WAIT_LIMIT_NS) { *s_abort = 1; latch_status(p.status, (int)MOQE_ERR_TIMEOUT); break; }
                        }
                    }
                    const float* src = p.partials + (size_t)(blockIdx.x + 1 + c0) * TOK * 128 + row;
                    float part[TOK];
#pragma unroll
                    for (int m = 0; m < TOK; ++m) part[m] = m < rows ? __ldcg(src + m * 128) : 0.f;
#pragma unroll
                    for (int m = 0; m < TOK; ++m) acc[m] += part[m];
                }
                // all 128 threads have seen the flags before any of them is cleared for the next call
                warrive(bar_esync);
                if (!wwait(bar_esync, esync_phase)) return false;
                esync_phase ^= 1u;
                if (*s_abort) return false;
                for (int i = et; i < n_others; i += 128) p.flags[blockIdx.x + 1 + i] = 0u;
                if (n < N) {
#pragma unroll
                    for (int m = 0; m < TOK; ++m)
                        if (m < rows) Y[(size_t)s_perm[j0 + m] * N + n] = __bfloat16_as_ushort(__float2bfloat16_rn(acc[m]));
                }
            }
            return true;
        };
        // Pieces before `upto` are complete as far as this warpgroup goes: hand its share over.
        auto flush_to = [&](int upto) -> bool {
            for (; flushed < upto; ++flushed) {
                const uint32_t par = (uint32_t)flushed & 1u;
                // every warpgroup has a slot of its own for its share, so none waits for another here -- only for the
                // last warpgroup to have read the previous piece's slots
                if (!wwait(bar_flushfree, par ^ 1u)) return false;
                const bool mine = acc_piece == flushed;
                float* slot = s_out + wg * (TOK * 128);
                if (wg != NWG - 1) {
#pragma unroll
                    for (int m = 0; m < TOK; ++m) slot[m * 128 + row] = mine ? acc[m] : 0.f;
                }
                warrive(bar_turn);
                if (wg == NWG - 1) {
                    // the last warpgroup adds the shares in warpgroup order (deterministic) once all have arrived
                    if (!wwait(bar_turn, par)) return false;
                    float total[TOK];
#pragma unroll
                    for (int m = 0; m < TOK; ++m) {
                        float v = s_out[m * 128 + row];
#pragma unroll
                        for (int u = 1; u < NWG - 1; ++u) v += s_out[u * (TOK * 128) + m * 128 + row];
                        total[m] = v + (mine ? acc[m] : 0.f);
                    }
                    warrive(bar_flushfree);
                    if (!finalize(flushed, total)) return false;
                }
                if (mine) {
#pragma unroll
                    for (int i = 0; i < TOK; ++i) acc[i] = 0.f;
                }
            }
            return true;
        };
        x_load(wg);
        int stg = wg % nstg, a = wg % NA;            // ring stage and A buffer of tile t, kept incrementally
        uint32_t wphase = (uint32_t)(wg / nstg) & 1u;
        for (int t = wg; ok && t < T; t += NWG) {
            const Tile ti(s_tile[t]);
            const ExpertSm& ex = s_ex[ti.e];
            // tile t - 6 is done, and so are all before it (MMAs are issued in tile order and a commit covers every
            // earlier one): A buffer t % 6 and token-tile stage (t + 4) % 10 are free, and the group that ended two
            // rounds ago (tile t - 8) can be drained without a wait of its own
            // First of all the warpgroup takes its turn for the pieces before the one its tile of two rounds ago
            // belongs to: all four warpgroups do this at the same distance behind their tiles and before they wait
            // for anything else, so none of them can be waiting for a tile that another holds back while it waits
            // for its turn.
            if (!(ok = flush_to(ph0))) break;
            if (!(ok = wait_done(t - NA))) break;
            x_load(t + NWG);
            drain(r0);
            r0 = r1;
            r1.t = -1;
            if (!(ok = wwait(bar_wfull + 8 * stg, wphase))) break;
            tc_fence_after();
            const unsigned char* stage = smem + L::ring_off + stg * stage_bytes;
            const int bits = ex.bits, group = ex.group, has_zeros = ex.has_zeros;
            // zero-point of this row for the tile: the tile's own meta, the per-channel array, or 2^(bits-1)
            float z = (float)(1 << (bits - 1));
            if (has_zeros)
                z = group == 0 ? __bfloat162float(p.ex[ti.e].zeros_pc[ti.nt * 128 + row])
                               : __bfloat162float(moqe_tile_zeros(stage, bits, 0)[row]);
            if (bits == 4) dequant_tile<4>(stage, row, pack_bf16x2(128.f + z, 128.f + z), lane_taddr + a * 64);
            else if (bits == 8) dequant_tile<8>(stage, row, pack_bf16x2(-z * 0.0001220703125f, -z * 0.0001220703125f), lane_taddr + a * 64);
            else dequant_tile<3>(stage, row, pack_bf16x2(128.f + z, 128.f + z), lane_taddr + a * 64);
            if (ti.ends()) {
                // the scale of the group that ends with this tile; its accumulator is drained two rounds later
                r1.t = t;
                r1.g = ti.g;
                r1.piece = ti.piece;
                r1.s = (group == 0 ? __half2float(p.ex[ti.e].scales_pc[ti.nt * 128 + row])
                                     : __half2float(moqe_tile_scales(stage, bits, has_zeros, 0)[row])) *
                         (bits == 8 ? W8_PRESCALE : 1.f);
            }
            warrive(bar_wempty + 8 * stg);
            asm volatile("cp.async.wait_group 1;" ::: "memory");      // this tile's token rows have landed
            fence_proxy_async();
            tmem_st_wait();
            tc_fence_before();
            warrive(bar_afull + 8 * a);
            ph0 = ph1;
            ph1 = ti.piece;
            last_t = t;
            stg += NWG;
            while (stg >= nstg) { stg -= nstg; wphase ^= 1u; }
            a += NWG;
            while (a >= NA) a -= NA;
        }
        if (ok) ok = flush_to(ph0);
        // the MMAs of this warpgroup's last tile (hence of all earlier ones) -- not of an older tile: a barrier of the
        // ring tells apart only tiles that are less than 8 apart
        if (ok && last_t >= 0) ok = wait_done(last_t);
        if (ok) {
            drain(r0);
            ok = flush_to(ph1);
        }
        if (ok) {
            drain(r1);
            flush_to(NP);
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*s_abort) {
        // let bulk copies that may still be in flight land before the shared memory is released
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == MMA_WARP) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

int g_dec_sm_count = 0;
int dec_sm_count() {
    if (!g_dec_sm_count) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&g_dec_sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (g_dec_sm_count <= 0) g_dec_sm_count = 148;
    }
    return g_dec_sm_count;
}

constexpr int DEC_MAX_GRID = 256;             // bound on CTAs the partial slots are sized for

// Relative cost of one packed tile in the work split (0 = its bytes).  Measured: an 8-bit tile is paced by its
// 16 KiB of HBM traffic, the narrower ones by the unpacking arithmetic, which is dearer per tile.
int g_dec_tile_cost[9] = {0, 0, 0, 11, 10, 0, 0, 0, 8};

}  // namespace

void decode_set_tile_cost(int bits, int cost) { if (bits >= 0 && bits <= 8 && cost >= 0) g_dec_tile_cost[bits] = cost; }

namespace {
// the work split of one call over `nl` layers of E experts each (pair index = layer * E + expert): costs, grid, and
// whether every CTA's tiles fit its tile table
bool decode_plan(const moqe_expert* const* ex, int nl, int E, DecSched& s, int& grid) {
    if (nl * E > MOQE_MAX_EXPERTS) return false;
    s.E = nl * E;
    s.C = 0;
    int wmax = 1, wmin = 1 << 30;
    for (int v = 0; v < nl * E; ++v) {
        const int cost = g_dec_tile_cost[ex[v]->bits];
        s.TT[v] = (ex[v]->Np / 128) * (ex[v]->Kp / 128);
        s.w[v] = cost > 0 ? cost : ex[v]->dev().tile_stride / 256;
        s.C += (long long)s.TT[v] * s.w[v];
        wmax = s.w[v] > wmax ? s.w[v] : wmax;
        wmin = s.w[v] < wmin ? s.w[v] : wmin;
    }
    // every CTA's cost share must be at least one tile of the dearest kind, so that every CTA between the owners of
    // a segment's first and last tile really owns a tile of it (the reduction counts them)
    grid = dec_sm_count();
    if (grid > DEC_MAX_GRID) grid = DEC_MAX_GRID;
    const long long work_items = s.C / wmax;
    if (work_items < grid) grid = work_items < 1 ? 1 : (int)work_items;
    s.G = grid;
    return s.C / grid / wmin + nl * E + 2 <= MAX_TILES;
}
bool formats_ok(const moqe_expert* const* ex, int n) {
    for (int v = 0; v < n; ++v)
        if (ex[v]->group != 0 && (ex[v]->group < 128 || ex[v]->group % 128 != 0)) return false;
    return true;
}
}  // namespace

bool decode_supported(int M, const moqe_expert* const* ex, int E) { return decode_supported_multi(M, ex, 1, E); }

bool decode_supported_multi(int M, const moqe_expert* const* ex, int nl, int E) {
    if (M > DECODE_MAX_ROWS || nl < 1 || nl * E > MOQE_MAX_EXPERTS || !formats_ok(ex, nl * E)) return false;
    DecSched s;
    int grid;
    return decode_plan(ex, nl, E, s, grid);
}

size_t decode_zero_bytes(int M, int Np) {
    if (M > DECODE_MAX_ROWS) return 0;
    (void)Np;
    return (size_t)DEC_MAX_GRID * sizeof(uint32_t);
}

size_t decode_workspace_bytes(int M, int Np, int E) {
    (void)E;
    if (M > DECODE_MAX_ROWS) return 0;
    const size_t counters = (decode_zero_bytes(M, Np) + 255) / 256 * 256;
    const size_t partials = (size_t)DEC_MAX_GRID * TOK * 128 * sizeof(float);
    return counters + partials;
}

moqe_status launch_qgemm_decode(const void* X, int M, int N, int K, const moqe_expert* const* ex, int E, void* Y,
                                const int32_t* perm, const int32_t* offsets, void* ws, size_t ws_bytes, cudaStream_t st) {
    (void)N; (void)K;
    return launch_qgemm_decode_multi(&X, M, 1, ex, E, &Y, perm, offsets, ws, ws_bytes, st);
}

// nl layers that share the routing; ex[l * E + e] = expert e of layer l; X[l] / Y[l] the layer's input / output
moqe_status launch_qgemm_decode_multi(const void* const* X, int M, int nl, const moqe_expert* const* ex, int E,
                                      void* const* Y, const int32_t* perm, const int32_t* offsets, void* ws,
                                      size_t ws_bytes, cudaStream_t st) {
    if (M == 0) return MOQE_OK;
    if (!decode_supported_multi(M, ex, nl, E)) return MOQE_ERR_UNSUPPORTED;
    DecParams p;
    int grid = 1;
    if (!decode_plan(ex, nl, E, p.sched, grid)) return MOQE_ERR_UNSUPPORTED;
    for (int l = 0; l < nl; ++l)
        for (int e = 0; e < E; ++e) {
            const int v = l * E + e;
            p.ex[v] = ex[v]->dev();
            p.X[v] = (const uint16_t*)X[l];
            p.Y[v] = (uint16_t*)Y[l];
            p.N[v] = ex[v]->N;
            p.K[v] = ex[v]->K;
            p.KB[v] = ex[v]->Kp / 128;
            p.rexp[v] = e;
        }
    if (!ws || ws_bytes < decode_workspace_bytes(M, ex[0]->Np, E)) return MOQE_ERR_WORKSPACE;
    p.flags = (uint32_t*)ws;
    p.partials = (float*)((char*)ws + (decode_zero_bytes(M, ex[0]->Np) + 255) / 256 * 256);
    p.perm = perm;
    p.offsets = offsets;
    p.M = M;
    p.R = E;
    p.status = device_status_word();
    static bool attr_set = false;
    cudaError_t err = cudaSuccess;
    if (!attr_set) {
        err = cudaFuncSetAttribute(qgemm_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DecSmem::dyn_bytes);
        attr_set = (err == cudaSuccess);
    }
    if (err == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid); cfg.blockDim = dim3(DEC_THREADS); cfg.dynamicSmemBytes = DecSmem::dyn_bytes; cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        err = cudaLaunchKernelEx(&cfg, qgemm_decode_kernel, p);
    }
    if (err != cudaSuccess) return MOQE_ERR_CUDA;
    count_launch();
    return cuda_ok(cudaGetLastError());
}

}  // namespace moqe
