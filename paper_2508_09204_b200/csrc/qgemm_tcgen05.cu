// Routed dequant-GEMM for large batches (prefill shapes): a persistent,
// warp-specialised grouped GEMM on the 5th-generation tensor cores.
//
//   tile         : 128 output channels (UMMA M, the TMEM lanes) x TN tokens (UMMA N, TMEM columns)
//   A operand    : the expert's weights.  Packed 128x128-code tiles arrive by bulk
//                  async copy; four "dequant" warps unpack them in registers to the
//                  exact integers (c - z) in bf16 and store them as a K-major,
//                  128-byte-swizzled shared-memory operand (64 k per stage).
//   B operand    : token rows, loaded by TMA (2-D tiled, 128-byte swizzle) from the
//                  expert-sorted activation matrix.
//   accumulation : tcgen05.mma (kind::f16, bf16 x bf16 -> fp32) into one of two TMEM
//                  buffers per quantization group; eight "epilogue" warps drain the
//                  finished buffer, multiply by the group's fp32 scale and add into
//                  register accumulators while the MMA fills the other buffer:
//                      Y[m][n] = sum_G s[n][G] * (sum_{k in G} X[m][k] * (c[n][k] - z[n][G]))
//                  so the tensor core only multiplies exactly representable numbers.
//                  Per-channel experts need a single scale at the end of K.
//   scheduling   : one CTA per SM walks the tile list (expert, token tile, channel
//                  tile) derived on the device from the per-expert offset table;
//                  rows are written straight to their original positions through
//                  `perm` (fused un-permutation).
//
// Every mbarrier wait is bounded (2 s of %globaltimer); on expiry the CTA sets
// an abort flag, latches MOQE_ERR_TIMEOUT, lets copies in flight land, frees
// its TMEM and returns.
//
// The operation is Section 3.1 of the paper (the selected quantization expert
// runs the sample); the paper describes no kernel.
#include <cuda.h>

#include <type_traits>

#include "dequant.cuh"
#include "ptx.cuh"
#include "tc_ptx.cuh"

namespace moqe {
namespace {

constexpr int TC_THREADS = 512;
constexpr int NS = 3;                 // operand stages (A tile + X tile, 64 k each)
constexpr int NWS = 3;                // packed-weight stages (128 k each)
constexpr int A_STAGE_BYTES = 128 * 128;          // 128 channels x 64 bf16
constexpr int W_STAGE_BYTES = 128 * 128 + 4 * 512;   // largest packed tile (W8 codes) + largest per-tile meta
constexpr int XBOX_ROWS = 64;
constexpr int XBOX_BYTES = XBOX_ROWS * 128;

struct TcParams {
    ExpertDev ex[MOQE_MAX_EXPERTS];
    const int32_t* perm;
    const int32_t* offsets;
    const int32_t* box_src;   // per 64-row box: first source row in X if its rows are consecutive there, else -1 (use Xp)
    uint16_t* Y;
    int* status;
    int M, N, K, Np, KB, E, n_tiles;
};

template <int TN>
struct Smem {
    static constexpr int a_off = 0;
    static constexpr int x_off = a_off + NS * A_STAGE_BYTES;
    static constexpr int w_off = x_off + NS * TN * 128;
    static constexpr int bar_off = w_off + NWS * W_STAGE_BYTES;
    // barriers: wfull[NWS] wempty[NWS] xfull[NS] afull[NS] empty[NS] accfull[2] accempty[2]
    static constexpr int n_bars = 2 * NWS + 3 * NS + 4;
    static constexpr int misc_off = bar_off + n_bars * 8;              // tmem addr, abort flag
    static constexpr int off_off = misc_off + 16;                      // offsets[E+1]
    static constexpr int perm_off = off_off + (MOQE_MAX_EXPERTS + 2) * 4;
    static constexpr int total = perm_off + 8 * (TN / 2) * 4;          // per epilogue warp: its columns' target rows
    static constexpr int dyn_bytes = total + 1024;                     // slack for manual 1024-byte alignment
};

// ---------------------------------------------------------------------------- TMA tile load
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

// ---------------------------------------------------------------------------- tile list
struct TileInfo { int e, nt, m0, rows; };

template <int TN>
__device__ __forceinline__ bool decode_tile(const int* s_off, int E, int n_tiles, int t, TileInfo& ti) {
    for (int e = 0; e < E; ++e) {
        int Me = s_off[e + 1] - s_off[e];
        int cnt = ((Me + TN - 1) / TN) * n_tiles;
        if (t < cnt) {
            int mt = t / n_tiles;
            ti.e = e;
            ti.nt = t - mt * n_tiles;
            ti.m0 = s_off[e] + mt * TN;
            ti.rows = min(TN, Me - mt * TN);
            return true;
        }
        t -= cnt;
    }
    return false;
}

// ---------------------------------------------------------------------------- dequant role
// One k-block (128 k) of one tile: wait for the packed tile, pull this thread's four pieces into
// registers, release the packed stage, then fill the two 64-k operand stages.
template <int BITS>
__device__ __forceinline__ bool dequant_kblock(const ExpertDev& ex, int nt, unsigned char* smem_w,
                                               unsigned char* smem_a_base, uint32_t bar_wfull, uint32_t bar_wempty,
                                               uint32_t wphase, uint32_t bar_empty0, uint32_t bar_afull0, Ring& ring,
                                               volatile int* abort_flag, int* status) {
    const int lane = threadIdx.x & 31, dw = (threadIdx.x >> 5) & 3;
    const int q = lane >> 3, r = (lane & 7) ^ (2 * q);          // slot = lane holds piece (q, r)
    constexpr int NWORDS = PieceWords<BITS>::n;
    const float sym_z = (float)(1 << (BITS - 1));
    // zero-points of the four pieces' channels, per chunk: per-channel experts read theirs from global memory
    // before the wait, the others from the tile's own meta once it has landed
    float z[4][4];
    const bool tile_zeros = ex.has_zeros && ex.group != 0;
#pragma unroll
    for (int pi = 0; pi < 4; ++pi) {
        const int n = nt * 128 + (2 * dw + (pi >> 1)) * 16 + (pi & 1) * 8 + r;
        const float v = (ex.has_zeros && ex.group == 0) ? __bfloat162float(ex.zeros_pc[n]) : sym_z;
#pragma unroll
        for (int G = 0; G < 4; ++G) z[pi][G] = v;
    }
    if (!mbar_wait(bar_wfull, wphase, abort_flag, status)) return false;
    uint32_t w[4][NWORDS];
#pragma unroll
    for (int pi = 0; pi < 4; ++pi)
        load_piece_smem<BITS>(smem_w + (2 * dw + (pi >> 1)) * moqe_blob_bytes(BITS), pi & 1, lane, w[pi]);
    if (tile_zeros) {
        const int per_tile = moqe_groups_per_tile(ex.group);
#pragma unroll
        for (int pi = 0; pi < 4; ++pi) {
            const int row = (2 * dw + (pi >> 1)) * 16 + (pi & 1) * 8 + r;
#pragma unroll
            for (int G = 0; G < 4; ++G) {
                const int j = per_tile == 4 ? G : (per_tile == 2 ? (G >> 1) : 0);
                z[pi][G] = __bfloat162float(moqe_tile_zeros(smem_w, BITS, j)[row]);
            }
        }
    }
    mbar_arrive(bar_wempty);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        if (!mbar_wait(bar_empty0 + 8 * ring.stage, ring.phase ^ 1u, abort_flag, status)) return false;
        unsigned char* a_stage = smem_a_base + ring.stage * A_STAGE_BYTES;
#pragma unroll
        for (int pi = 0; pi < 4; ++pi) {
            const int row = (2 * dw + (pi >> 1)) * 16 + (pi & 1) * 8 + r;
            auto put = [&](auto Gc) {
                constexpr int G = decltype(Gc)::value;
                uint32_t out[4];
                unpack_chunk<BITS, G>(w[pi], z[pi][G], out);
                const int chunk = (G & 1) * 4 + q;
                *reinterpret_cast<uint4*>(a_stage + row * 128 + ((chunk ^ (row & 7)) << 4)) =
                    make_uint4(out[0], out[1], out[2], out[3]);
            };
            if (h == 0) { put(std::integral_constant<int, 0>{}); put(std::integral_constant<int, 1>{}); }
            else        { put(std::integral_constant<int, 2>{}); put(std::integral_constant<int, 3>{}); }
        }
        fence_proxy_async();
        mbar_arrive(bar_afull0 + 8 * ring.stage);
        ring.advance(NS);
    }
    return true;
}

// ---------------------------------------------------------------------------- the kernel
// W2: the instantiation that also takes 2-bit experts (kept apart: the extra unpack path costs the dequant warps of
// the common instantiation 14 % through register allocation alone)
template <int TN, bool REGSPLIT, bool W2>
__global__ void __launch_bounds__(TC_THREADS, 1) qgemm_tc_kernel(const __grid_constant__ TcParams p,
                                                                const __grid_constant__ CUtensorMap tmap,
                                                                const __grid_constant__ CUtensorMap tmap_x) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    using L = Smem<TN>;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + L::bar_off;
    const uint32_t bar_wfull = bar0, bar_wempty = bar0 + 8 * NWS, bar_xfull = bar0 + 16 * NWS;
    const uint32_t bar_afull = bar_xfull + 8 * NS, bar_empty = bar_afull + 8 * NS;
    const uint32_t bar_accfull = bar_empty + 8 * NS, bar_accempty = bar_accfull + 16;
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + L::misc_off);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::misc_off + 4);
    int* s_off = reinterpret_cast<int*>(smem + L::off_off);
    int* s_perm = reinterpret_cast<int*>(smem + L::perm_off);

    if (tid == 0) {
        for (int i = 0; i < NWS; ++i) { mbar_init(bar_wfull + 8 * i, 1); mbar_init(bar_wempty + 8 * i, 128); }
        for (int i = 0; i < NS; ++i) { mbar_init(bar_xfull + 8 * i, 1); mbar_init(bar_afull + 8 * i, 128); mbar_init(bar_empty + 8 * i, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar_accfull + 8 * i, 1); mbar_init(bar_accempty + 8 * i, 256); }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i <= p.E; i += TC_THREADS) s_off[i] = p.offsets[i];
    if (warp == 1) tmem_alloc(sbase + L::misc_off, 2 * TN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem;

    if (warp < 4) {
        if constexpr (REGSPLIT) asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        if (warp == 0 && lane == 0) {
            // ---------------- X producer: TMA boxes of 64 token rows x 64 k ----------------
            Ring ring;
            TileInfo ti;
            bool ok = true;
            for (int t = blockIdx.x; ok && decode_tile<TN>(s_off, p.E, p.n_tiles, t, ti); t += gridDim.x) {
                const int nbox = (ti.rows + XBOX_ROWS - 1) / XBOX_ROWS;
                // where each 64-row box of this tile comes from: straight from X when its rows are consecutive there
                int box0 = (ti.m0 - s_off[ti.e]) / XBOX_ROWS;
                for (int e2 = 0; e2 < ti.e; ++e2) box0 += (s_off[e2 + 1] - s_off[e2] + XBOX_ROWS - 1) / XBOX_ROWS;
                int src_row[TN / XBOX_ROWS];
#pragma unroll
                for (int b = 0; b < TN / XBOX_ROWS; ++b) src_row[b] = b < nbox ? p.box_src[box0 + b] : -1;
                for (int ks = 0; ks < 2 * p.KB; ++ks) {
                    if (!(ok = mbar_wait(bar_empty + 8 * ring.stage, ring.phase ^ 1u, s_abort, p.status))) break;
                    const uint32_t full = bar_xfull + 8 * ring.stage;
                    mbar_expect_tx(full, nbox * XBOX_BYTES);
                    const uint32_t dst = sbase + L::x_off + ring.stage * (TN * 128);
#pragma unroll
                    for (int b = 0; b < TN / XBOX_ROWS; ++b) {
                        if (b < nbox) {
                            if (src_row[b] >= 0) tma_load_2d(dst + b * XBOX_BYTES, &tmap_x, ks * 64, src_row[b], full);
                            else tma_load_2d(dst + b * XBOX_BYTES, &tmap, ks * 64, ti.m0 + b * XBOX_ROWS, full);
                        }
                    }
                    ring.advance(NS);
                }
            }
        } else if (warp == 2 && lane == 0) {
            // ---------------- W producer: one packed 128x128-code tile per k-block ----------------
            Ring ring;
            TileInfo ti;
            bool ok = true;
            for (int t = blockIdx.x; ok && decode_tile<TN>(s_off, p.E, p.n_tiles, t, ti); t += gridDim.x) {
                const ExpertDev& ex = p.ex[ti.e];
                const uint32_t bytes = (uint32_t)ex.tile_stride;          // codes + the tile's scales / zero-points
                const uint8_t* src = ex.tiles + (size_t)ti.nt * p.KB * bytes;
                for (int kb = 0; kb < p.KB; ++kb) {
                    if (!(ok = mbar_wait(bar_wempty + 8 * ring.stage, ring.phase ^ 1u, s_abort, p.status))) break;
                    const uint32_t full = bar_wfull + 8 * ring.stage;
                    mbar_expect_tx(full, bytes);
                    bulk_load(sbase + L::w_off + ring.stage * W_STAGE_BYTES, src + (size_t)kb * bytes, bytes, full);
                    ring.advance(NWS);
                }
            }
        } else if (warp == 1) {
            // ---------------- MMA issuer ----------------
            // (Its waits spin on the plain try_wait: they sit on the critical path and coming round a short spin is
            // faster than waking from the hinted sleep.)
            // The WHOLE warp walks the tiles, so that control flow stays warp-uniform, and one elected lane issues
            // straight-line MMAs whose operands were all computed beforehand.  Measured on B200: issued this way a
            // 128x256x16 MMA costs its 128 tensor-pipe cycles (and a 16-column one 24); issued from a loop that
            // only lane 0 runs (`if (lane == 0)`) and that builds descriptors between MMAs, every MMA costs ~250.
            Ring ring;
            TileInfo ti;
            bool ok = true;
            uint32_t acc_use[2] = {0, 0};
            int buf = 0;
            for (int t = blockIdx.x; ok && decode_tile<TN>(s_off, p.E, p.n_tiles, t, ti); t += gridDim.x) {
                const ExpertDev& ex = p.ex[ti.e];
                const int n_eff = (ti.rows + 15) & ~15;
                const uint32_t idesc = umma_idesc(n_eff);
                const int group_k = ex.group == 0 ? p.KB * 128 : min(ex.group, 128);
                int kcount = 0;
                for (int ks = 0; ok && ks < 2 * p.KB; ++ks) {
                    if (!(ok = __all_sync(0xffffffffu, mbar_wait_short(bar_xfull + 8 * ring.stage, ring.phase, s_abort, p.status)))) break;
                    if (!(ok = __all_sync(0xffffffffu, mbar_wait_short(bar_afull + 8 * ring.stage, ring.phase, s_abort, p.status)))) break;
                    const uint64_t adesc = umma_desc_sw128(sbase + L::a_off + ring.stage * A_STAGE_BYTES);
                    const uint64_t bdesc = umma_desc_sw128(sbase + L::x_off + ring.stage * (TN * 128));
                    const uint32_t empty_bar = bar_empty + 8 * ring.stage;
                    if (group_k >= 64) {
                        // the stage's four MMAs feed one accumulator buffer
                        if (kcount == 0 &&
                            !(ok = __all_sync(0xffffffffu, mbar_wait_short(bar_accempty + 8 * buf, (acc_use[buf] & 1u) ^ 1u, s_abort, p.status)))) break;
                        tc_fence_after();
                        const uint32_t d = tmem_base + buf * TN;
                        const bool group_ends = kcount + 64 == group_k;
                        if (elect_one()) {
                            umma_bf16(d, adesc, bdesc, idesc, kcount > 0 ? 1u : 0u);
                            umma_bf16(d, adesc + 2, bdesc + 2, idesc, 1u);
                            umma_bf16(d, adesc + 4, bdesc + 4, idesc, 1u);
                            umma_bf16(d, adesc + 6, bdesc + 6, idesc, 1u);
                            if (group_ends) umma_commit(bar_accfull + 8 * buf);
                            umma_commit(empty_bar);
                        }
                        __syncwarp();
                        kcount += 64;
                        if (group_ends) {
                            acc_use[buf]++;
                            buf ^= 1;
                            kcount = 0;
                        }
                    } else {
                        // groups of 32 k: two accumulator buffers per stage
                        tc_fence_after();
                        for (int j = 0; ok && j < 4; ++j) {
                            if (kcount == 0) {
                                if (!(ok = __all_sync(0xffffffffu, mbar_wait_short(bar_accempty + 8 * buf, (acc_use[buf] & 1u) ^ 1u, s_abort, p.status)))) break;
                                tc_fence_after();
                            }
                            const bool group_ends = kcount + 16 == group_k;
                            if (elect_one()) {
                                umma_bf16(tmem_base + buf * TN, adesc + 2 * j, bdesc + 2 * j, idesc, kcount > 0 ? 1u : 0u);
                                if (group_ends) umma_commit(bar_accfull + 8 * buf);
                                if (j == 3) umma_commit(empty_bar);
                            }
                            __syncwarp();
                            kcount += 16;
                            if (group_ends) {
                                acc_use[buf]++;
                                buf ^= 1;
                                kcount = 0;
                            }
                        }
                        if (!ok) break;
                    }
                    ring.advance(NS);
                }
            }
        }
    } else if (warp < 8) {
        if constexpr (REGSPLIT) asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
        // ---------------- dequant warps ----------------
        Ring wring, ring;
        TileInfo ti;
        bool ok = true;
        for (int t = blockIdx.x; ok && decode_tile<TN>(s_off, p.E, p.n_tiles, t, ti); t += gridDim.x) {
            const ExpertDev& ex = p.ex[ti.e];
            for (int kb = 0; ok && kb < p.KB; ++kb) {
                unsigned char* sw = smem + L::w_off + wring.stage * W_STAGE_BYTES;
                const uint32_t wf = bar_wfull + 8 * wring.stage, we = bar_wempty + 8 * wring.stage;
                if (ex.bits == 4)
                    ok = dequant_kblock<4>(ex, ti.nt, sw, smem + L::a_off, wf, we, wring.phase, bar_empty, bar_afull, ring, s_abort, p.status);
                else if (ex.bits == 8)
                    ok = dequant_kblock<8>(ex, ti.nt, sw, smem + L::a_off, wf, we, wring.phase, bar_empty, bar_afull, ring, s_abort, p.status);
                else if (W2 && ex.bits == 2) {
                    if constexpr (W2)
                        ok = dequant_kblock<2>(ex, ti.nt, sw, smem + L::a_off, wf, we, wring.phase, bar_empty, bar_afull, ring, s_abort, p.status);
                } else
                    ok = dequant_kblock<3>(ex, ti.nt, sw, smem + L::a_off, wf, we, wring.phase, bar_empty, bar_afull, ring, s_abort, p.status);
                wring.advance(NWS);
            }
        }
    } else {
        if constexpr (REGSPLIT) asm volatile("setmaxnreg.inc.sync.aligned.u32 184;");
        // ---------------- epilogue warps: scale-and-accumulate, then store ----------------
        constexpr int NCOL = TN / 2;                       // columns (tokens) per warp
        const int ew = warp - 8, quarter = ew & 3, colhalf = ew >> 2;
        const int col0 = colhalf * NCOL;
        const int row = quarter * 32 + lane;               // channel inside the tile = TMEM lane
        TileInfo ti;
        bool ok = true;
        uint32_t acc_use[2] = {0, 0};
        int buf = 0;
        for (int t = blockIdx.x; ok && decode_tile<TN>(s_off, p.E, p.n_tiles, t, ti); t += gridDim.x) {
            const ExpertDev& ex = p.ex[ti.e];
            const int n = ti.nt * 128 + row;
            const int n_eff = (ti.rows + 15) & ~15;
            int* my_perm = s_perm + ew * NCOL;                     // private to this warp: no cross-warp barrier
            __syncwarp();
            for (int i = lane; i < NCOL; i += 32) my_perm[i] = (col0 + i < ti.rows) ? p.perm[ti.m0 + col0 + i] : -1;
            __syncwarp();
            float acc[NCOL];
#pragma unroll
            for (int i = 0; i < NCOL; ++i) acc[i] = 0.f;
            const int group_k = ex.group == 0 ? p.KB * 128 : min(ex.group, 128);
            const int ngroups = p.KB * 128 / group_k;
            for (int gi = 0; ok && gi < ngroups; ++gi) {
                float s;
                if (ex.group == 0) {
                    s = __half2float(ex.scales_pc[n]);
                } else {                                   // the scale sits in the meta of the tile the group lies in
                    const int per_tile = moqe_groups_per_tile(ex.group);
                    const unsigned char* tile = ex.tiles + ((size_t)ti.nt * p.KB + gi / per_tile) * (size_t)ex.tile_stride;
                    s = __half2float(moqe_tile_scales(tile, ex.bits, ex.has_zeros, gi % per_tile)[row]);
                }
                if (ex.bits == 8) s *= W8_PRESCALE;          // 8-bit chunks are unpacked as (c - z) * 2^-13
                if (!(ok = mbar_wait(bar_accfull + 8 * buf, acc_use[buf] & 1u, s_abort, p.status))) break;
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < NCOL / 32; ++c) {
                    if (col0 + c * 32 < n_eff) {
                        uint32_t v[32];
                        tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * TN + col0 + c * 32, v);
                        tmem_ld_wait();
                        // acc += s * v, two columns per instruction (each half rounds as a scalar fma does)
#pragma unroll
                        for (int i = 0; i < 32; i += 2)
                            asm("{\n\t.reg .b64 a, x, s2;\n\tmov.b64 a, {%0, %1};\n\tmov.b64 x, {%3, %4};\n\tmov.b64 s2, {%2, %2};\n\t"
                                "fma.rn.f32x2 a, s2, x, a;\n\tmov.b64 {%0, %1}, a;\n\t}"
                                : "+f"(acc[c * 32 + i]), "+f"(acc[c * 32 + i + 1]) : "f"(s), "r"(v[i]), "r"(v[i + 1]));
                    }
                }
                tc_fence_before();
                mbar_arrive(bar_accempty + 8 * buf);
                acc_use[buf]++;
                buf ^= 1;
            }
            if (ok && n < p.N) {
#pragma unroll
                for (int i = 0; i < NCOL; ++i) {
                    const int col = col0 + i;
                    if (col < ti.rows) p.Y[(size_t)my_perm[i] * p.N + n] = __bfloat16_as_ushort(__float2bfloat16_rn(acc[i]));
                }
            }
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (*s_abort) {
        // let bulk copies that may still be in flight land before the shared memory is released
        unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 2 * TN);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)f;
    }
    return fn;
}

int g_tile_tokens_override = 0;

}  // namespace

void tc_set_tile_tokens(int tn) { g_tile_tokens_override = tn; }

size_t tc_workspace_bytes(int M, int K, int E, int Np) {
    (void)Np;
    return ((size_t)M * K * 2 + 255) / 256 * 256 + gather_boxes_bytes(M, E);
}

moqe_status launch_qgemm_tc(const void* X, int M, int N, int K, const moqe_expert* const* ex, int E, void* Y,
                            const int32_t* perm, const int32_t* offsets, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (M == 0) return MOQE_OK;
    if (!ws || ws_bytes < tc_workspace_bytes(M, K, E, ex[0]->Np)) return MOQE_ERR_WORKSPACE;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return MOQE_ERR_CUDA;
    // 1. expert-sorted copy of the activations (rows with an invalid id become zero rows at the end)
    void* Xp = ws;
    int32_t* box_src = (int32_t*)((char*)ws + ((size_t)M * K * 2 + 255) / 256 * 256);
    moqe_status s = launch_gather_boxes(X, perm, offsets, M, K, E, Xp, box_src, st);
    if (s != MOQE_OK) return s;
    // 2. tensor map over Xp[M][K] bf16: boxes of 64 k x 64 rows, 128-byte swizzle, zero fill outside
    CUtensorMap tmap;
    cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)M};
    cuuint64_t gstride[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)XBOX_ROWS};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Xp, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return MOQE_ERR_CUDA;
    CUtensorMap tmap_x;                                   // the same boxes over the caller's X (unsorted rows)
    if (enc(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(X), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return MOQE_ERR_CUDA;
    TcParams p;
    for (int e = 0; e < E; ++e) {
        p.ex[e] = ex[e]->dev();
    }
    p.box_src = box_src;
    p.perm = perm; p.offsets = offsets; p.Y = (uint16_t*)Y; p.status = device_status_word();
    p.M = M; p.N = N; p.K = K; p.Np = ex[0]->Np; p.KB = ex[0]->Kp / 128; p.E = E; p.n_tiles = p.Np / 128;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int tn = g_tile_tokens_override ? g_tile_tokens_override : (M >= 2048 ? 256 : 128);
    long long max_tiles = ((long long)(M + tn - 1) / tn + E) * p.n_tiles;
    int grid = (int)(max_tiles < sms ? max_tiles : sms);
    cudaError_t err;
    bool any_w2 = false;
    for (int e = 0; e < E; ++e) any_w2 = any_w2 || ex[e]->bits == 2;
    // (the attribute is set at every launch: it belongs to the current device, and the call is cheap)
    auto launch = [&](auto kernel, int smem) -> bool {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
        kernel<<<grid, TC_THREADS, smem, st>>>(p, tmap, tmap_x);
        return true;
    };
    bool launched;
    if (tn == 256)
        launched = any_w2 ? launch(qgemm_tc_kernel<256, true, true>, Smem<256>::dyn_bytes) : launch(qgemm_tc_kernel<256, true, false>, Smem<256>::dyn_bytes);
    else
        launched = any_w2 ? launch(qgemm_tc_kernel<128, false, true>, Smem<128>::dyn_bytes) : launch(qgemm_tc_kernel<128, false, false>, Smem<128>::dyn_bytes);
    if (!launched) return MOQE_ERR_CUDA;
    err = cudaGetLastError();
    count_launch();
    return cuda_ok(err);
}

}  // namespace moqe
