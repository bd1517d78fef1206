// Routed GEMM for large batches on layers with SMALL weights (the 1x1 convolutions of a CNN: a few hundred
// kilobytes per expert).  Such a layer is bound by its activations -- M*(K+N)*2 bytes against N*K*b/8 -- so the
// kernel is built around streaming X and Y: each expert's weights are first expanded to a plain bf16 matrix
// (launch_dense_unpack; they stay in L2), and a persistent, warp-specialised tcgen05 GEMM then runs with the TOKENS as
// the 128 rows of the MMA:
//
//   tile      : 128 token rows of one expert x up to 256 output channels (one TMEM accumulator of up to 256 columns,
//               two of them so that the epilogue of a tile overlaps the MMAs of the next)
//   operands  : 64 k per stage.  The channel rows of the dense weights by TMA (2-D tiled, 128-byte swizzle, no
//               multicast); the token rows in boxes of 64 rows: by TMA straight from X where the box's sorted rows are
//               consecutive there (always, for per-image routing of whole 64-row runs), else gathered row by row
//               through `perm` by the producer warp's 16-byte cp.async copies into the same swizzled layout -- the
//               fused permutation, no gathered copy of X exists
//   epilogue  : one thread per token row reads its accumulator row from TMEM, multiplies by the per-channel scale,
//               rounds to bf16 and writes up to 512 contiguous bytes of Y at the row's ORIGINAL position (fused
//               un-permutation).  X is read once per channel chunk and Y written once.
//
// Per-channel experts reach the tensor core as the exact integers c - z (scale applied to the fp32 sums).  Grouped
// experts as TWO bf16 numbers per weight, hi + lo = s * (c - z) to 2^-17, and the k loop runs over both halves (the
// token stage is fetched again from L2 for the second half): twice the tensor work on a path the tensor cores do not
// bound, and no rounding of weights that the tolerance of the routed product would see.
//
// Every mbarrier wait is bounded; on expiry the CTA raises its abort flag, latches MOQE_ERR_TIMEOUT, lets copies in
// flight land, frees its TMEM and returns.
//
// The operation is Section 3.1 of the paper (the selected quantization expert runs the sample); the paper describes
// no kernel.
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tc_ptx.cuh"

namespace moqe {
namespace {

constexpr int DN_THREADS = 416;                 // warp 0: producer (TMA + gather), warp 1: MMA issuer, warps 2..9: epilogue,
                                                // warps 10..12: gather helpers
constexpr int DN_GATHER_WARPS = 4;              // warp 0 and the helpers
constexpr int DN_EPI_THREADS = 256;
constexpr int DN_MAX_STAGES = 8;
constexpr int DN_XSTAGE = 128 * 128;            // 128 token rows x 64 k bf16
constexpr int DN_NC = 256;                      // channels per accumulator
constexpr int DN_MAX_K = 1024;
constexpr int DN_POOL_BYTES = 216 * 1024;       // staged output rows + resident weights + operand stages, split at run time
constexpr int DN_WRES_MAX = 64 * 1024;          // an expert's dense weights stay in shared memory when they are this small

struct DnSmem {
    static constexpr int pool_off = 0;                                     // [staged output rows][resident weights][stages]
    static constexpr int cs_off = DN_POOL_BYTES;                           // column scales of the epilogue's expert
    static constexpr int bar_off = cs_off + 1024 * 4;
    static constexpr int n_bars = 2 * DN_MAX_STAGES + 6;                   // full[8] empty[8] accfull[2] accempty[2] wres_full wres_empty
    static constexpr int misc_off = bar_off + n_bars * 8;
    static constexpr int off_off = misc_off + 16;
    static constexpr int total = off_off + (MOQE_MAX_EXPERTS + 2) * 4;
    static constexpr int dyn_bytes = total + 1024;
};

struct DnParams {
    const int32_t* perm;
    const int32_t* offsets;
    const uint16_t* X;          // token rows [M][K] bf16, unsorted
    const float* col_scale;     // [E][Np]
    uint16_t* Y;
    int* status;
    int M, N, K, Np, Kp, E, Ksteps;   // Ksteps: 64-k stages that hold real k (columns beyond K read as zeros)
    int Nw;                        // channel rows that take part: N rounded up to whole 64-row boxes
    unsigned split_mask;           // bit e: expert e is stored as hi + lo halves (grouped formats)
    int resident, max_steps;       // the experts' dense weights fit shared memory; 64-k steps of the largest one
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

struct DnTile { int e, m0, rows, box0; };
// token tile t of the call: expert, first sorted row, rows, index of its first 64-row box
__device__ __forceinline__ bool dn_tile(const int* s_off, int E, int t, DnTile& ti) {
    int box0 = 0;
    for (int e = 0; e < E; ++e) {
        const int Me = s_off[e + 1] - s_off[e];
        const int cnt = (Me + 127) / 128;
        if (t < cnt) {
            ti.e = e;
            ti.m0 = s_off[e] + t * 128;
            ti.rows = min(128, Me - t * 128);
            ti.box0 = box0 + 2 * t;
            return true;
        }
        t -= cnt;
        box0 += (Me + 63) / 64;
    }
    return false;
}

__global__ void __launch_bounds__(DN_THREADS, 1) qgemm_dense_kernel(const __grid_constant__ DnParams p,
                                                                    const __grid_constant__ CUtensorMap tmap_x,
                                                                    const __grid_constant__ CUtensorMap tmap_w) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    using L = DnSmem;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_full = sbase + L::bar_off, bar_empty = bar_full + 8 * DN_MAX_STAGES;
    const uint32_t bar_accfull = bar_empty + 8 * DN_MAX_STAGES, bar_accempty = bar_accfull + 16;
    const uint32_t bar_wres_full = bar_accempty + 16, bar_wres_empty = bar_wres_full + 8;
    // Shared-memory plan.  Output rows are staged with a padded pitch; an expert's dense weights stay resident when all
    // their 64-k steps fit DN_WRES_MAX (the token rows are then the only stream); the rest is cut into operand stages of
    // 128 token rows (+ the channel rows of one accumulator when the weights are streamed too).
    const int nc_rows = min(DN_NC, p.Nw);
    const int out_pitch = nc_rows * 2 + 16;
    const int out_bytes = (128 * out_pitch + 1023) & ~1023;
    const int wres_bytes = p.resident ? p.max_steps * p.Nw * 128 : 0;
    const int stage_bytes = DN_XSTAGE + (p.resident ? 0 : nc_rows * 128);
    const int nstg = min(DN_MAX_STAGES, (DN_POOL_BYTES - out_bytes - wres_bytes) / stage_bytes);
    const uint32_t out_base = sbase + L::pool_off, wres_base = out_base + out_bytes, ring_base = wres_base + wres_bytes;
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + L::misc_off);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::misc_off + 4);
    int* s_off = reinterpret_cast<int*>(smem + L::off_off);
    float* s_cs = reinterpret_cast<float*>(smem + L::cs_off);

    if (tid == 0) {
        for (int i = 0; i < DN_MAX_STAGES; ++i) { mbar_init(bar_full + 8 * i, 1 + 32 * DN_GATHER_WARPS); mbar_init(bar_empty + 8 * i, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar_accfull + 8 * i, 1); mbar_init(bar_accempty + 8 * i, DN_EPI_THREADS); }
        mbar_init(bar_wres_full, 1);
        mbar_init(bar_wres_empty, 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i <= p.E; i += DN_THREADS) s_off[i] = p.offsets[i];
    if (warp == 1) tmem_alloc(sbase + L::misc_off, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem;
    const int nchunks = (p.Nw + DN_NC - 1) / DN_NC, kstages = p.Ksteps;

    if (warp == 0 || warp >= 10) {
        // ---------------- producers: token boxes and weight boxes, 64 k per stage ----------------
        // Four warps walk the tiles in step.  Lane 0 of warp 0 issues the TMA copies: the weight boxes, and every 64-row
        // token box whose sorted rows are consecutive in X (always, for per-image routing of whole 64-row runs) straight
        // from X.  A box whose rows are scattered in X is gathered by the 128 lanes with 16-byte cp.async copies, row by
        // row through `perm`, into the same 128-byte-swizzled layout (warp g takes box rows 16g .. 16g + 15); a
        // stage's full barrier takes one arrival per lane (tied to the lane's copies where it made some) on top of
        // the transaction count.
        const int g = warp == 0 ? 0 : warp - 9;
        const bool tma_lane = warp == 0 && lane == 0;
        Ring ring;
        DnTile ti;
        bool ok = true;
        int w_e = -1;
        uint32_t w_uses = 0;
        // this lane's entries of `perm` for the tile's rows lane, lane + 32, lane + 64, lane + 96 (-1 beyond the tile),
        // fetched one tile ahead: a global round trip per tile would otherwise sit in front of every tile's copies
        auto fetch_rows = [&](const DnTile& t, int (&o)[4]) {
#pragma unroll
            for (int q = 0; q < 4; ++q) o[q] = q * 32 + lane < t.rows ? p.perm[t.m0 + q * 32 + lane] : -1;
        };
        DnTile nx;
        int npv[4] = {-1, -1, -1, -1};
        bool have = dn_tile(s_off, p.E, blockIdx.x, nx);
        if (have) fetch_rows(nx, npv);
        const uint16_t* Xg = p.X;
        for (int t = blockIdx.x; ok && have; t += gridDim.x) {
            ti = nx;
            const int pv[4] = {npv[0], npv[1], npv[2], npv[3]};
            have = dn_tile(s_off, p.E, t + gridDim.x, nx);
            if (have) fetch_rows(nx, npv);
            const int nbox = (ti.rows + 63) / 64;
            int src_row[2];                 // first row in X of a box whose rows are consecutive there, else -1
            int xr[2][4];                   // the X row of box row 16g + 4i + lane / 8 (-1: none, zero fill)
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                const int cnt = min(64, ti.rows - 64 * b);
                const int first = __shfl_sync(0xffffffffu, pv[2 * b], 0);
                const bool mine = (lane >= cnt || pv[2 * b] == first + lane) && (lane + 32 >= cnt || pv[2 * b + 1] == first + lane + 32);
                src_row[b] = (b < nbox && __all_sync(0xffffffffu, mine)) ? first : -1;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    xr[b][i] = __shfl_sync(0xffffffffu, g < 2 ? pv[2 * b] : pv[2 * b + 1], (16 * g + 4 * i + (lane >> 3)) & 31);
            }
            const bool gather0 = nbox > 0 && src_row[0] < 0, gather1 = nbox > 1 && src_row[1] < 0;
            const int n_tma = (nbox > 0 && !gather0 ? 1 : 0) + (nbox > 1 && !gather1 ? 1 : 0);
            const int steps = ((p.split_mask >> ti.e) & 1u) ? 2 * kstages : kstages;
            if (warp == 0 && p.resident && ti.e != w_e) {
                // a new expert: its dense weights replace the resident ones once the MMAs that read those are done
                if (w_uses > 0 && !(ok = __all_sync(0xffffffffu, mbar_wait(bar_wres_empty, (w_uses - 1) & 1u, s_abort, p.status)))) break;
                if (lane == 0) {
                    mbar_expect_tx(bar_wres_full, (uint32_t)(steps * (p.Nw / 64)) * 8192u);
                    for (int ks = 0; ks < steps; ++ks) {
                        const int wcol = ks < kstages ? ks * 64 : p.Kp + (ks - kstages) * 64;
                        for (int b = 0; b < p.Nw / 64; ++b)
                            tma_load_2d(wres_base + (ks * (p.Nw / 64) + b) * 8192, &tmap_w, wcol, ti.e * p.Np + b * 64, bar_wres_full);
                    }
                }
                w_e = ti.e;
                ++w_uses;
            }
            for (int nc = 0; ok && nc < nchunks; ++nc) {
                const int wrows = min(DN_NC, p.Nw - nc * DN_NC);
                for (int ks = 0; ks < steps; ++ks) {
                    if (!(ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * ring.stage, ring.phase ^ 1u, s_abort, p.status)))) break;
                    const uint32_t full = bar_full + 8 * ring.stage;
                    const uint32_t xd = ring_base + ring.stage * stage_bytes;
                    const int xcol = (ks < kstages ? ks : ks - kstages) * 64;             // the second half re-reads the tokens
                    if (tma_lane) {
                        mbar_expect_tx(full, (uint32_t)(n_tma + (p.resident ? 0 : wrows / 64)) * 8192u);
                        if (nbox > 0 && !gather0) tma_load_2d(xd, &tmap_x, xcol, src_row[0], full);
                        if (nbox > 1 && !gather1) tma_load_2d(xd + 8192, &tmap_x, xcol, src_row[1], full);
                        if (!p.resident) {
                            const int wcol = ks < kstages ? ks * 64 : p.Kp + (ks - kstages) * 64;
                            const uint32_t wd = xd + DN_XSTAGE;
                            for (int b = 0; b < wrows / 64; ++b)
                                tma_load_2d(wd + b * 8192, &tmap_w, wcol, ti.e * p.Np + nc * DN_NC + b * 64, full);
                        }
                    }
                    if (gather0 || gather1) {
                        const int chunk = lane & 7, kk = xcol + chunk * 8;
#pragma unroll
                        for (int b = 0; b < 2; ++b) {
                            if (b == 0 ? gather0 : gather1) {
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const int r = 16 * g + 4 * i + (lane >> 3);
                                    const bool real = xr[b][i] >= 0 && kk < p.K;
                                    const uint16_t* src = real ? Xg + (size_t)xr[b][i] * p.K + kk : Xg;
                                    const uint32_t dst = xd + b * 8192 + r * 128 + ((chunk ^ (r & 7)) << 4);
                                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(real ? 16 : 0) : "memory");
                                }
                            }
                        }
                        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(full) : "memory");
                    } else {
                        mbar_arrive(full);
                    }
                    ring.advance(nstg);
                }
            }
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
    } else if (warp == 1) {
        // ---------------- MMA issuer: the whole warp walks the tiles, one elected lane issues ----------------
        Ring ring;
        DnTile ti;
        bool ok = true;
        uint32_t acc_use[2] = {0, 0};
        int buf = 0, w_e = -1;
        uint32_t w_uses = 0;
        for (int t = blockIdx.x; ok && dn_tile(s_off, p.E, t, ti); t += gridDim.x) {
            if (p.resident && ti.e != w_e) {
                // hand the resident weights of the previous expert back (when every MMA issued so far is done) and
                // wait for the new expert's
                if (w_uses > 0) {
                    if (elect_one()) umma_commit(bar_wres_empty);
                    __syncwarp();
                }
                if (!(ok = __all_sync(0xffffffffu, mbar_wait(bar_wres_full, w_uses & 1u, s_abort, p.status)))) break;
                w_e = ti.e;
                ++w_uses;
            }
            for (int nc = 0; ok && nc < nchunks; ++nc) {
                const int wrows = min(DN_NC, p.Nw - nc * DN_NC);
                const uint32_t idesc = umma_idesc(wrows);
                if (!(ok = __all_sync(0xffffffffu, mbar_wait(bar_accempty + 8 * buf, (acc_use[buf] & 1u) ^ 1u, s_abort, p.status)))) break;
                const uint32_t d = tmem_base + buf * DN_NC;
                const int steps = ((p.split_mask >> ti.e) & 1u) ? 2 * kstages : kstages;
                for (int ks = 0; ks < steps; ++ks) {
                    if (!(ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * ring.stage, ring.phase, s_abort, p.status)))) break;
                    fence_proxy_async();                 // gathered token rows were written by plain (generic-proxy) copies
                    tc_fence_after();
                    const uint32_t stage = ring_base + ring.stage * stage_bytes;
                    const uint64_t adesc = umma_desc_sw128(stage);
                    const uint64_t bdesc = umma_desc_sw128(p.resident ? wres_base + ks * p.Nw * 128 + nc * DN_NC * 128 : stage + DN_XSTAGE);
                    const uint32_t empty_bar = bar_empty + 8 * ring.stage;
                    const bool last = ks + 1 == steps;
                    if (elect_one()) {
                        umma_bf16(d, adesc, bdesc, idesc, ks > 0 ? 1u : 0u);
                        umma_bf16(d, adesc + 2, bdesc + 2, idesc, 1u);
                        umma_bf16(d, adesc + 4, bdesc + 4, idesc, 1u);
                        umma_bf16(d, adesc + 6, bdesc + 6, idesc, 1u);
                        umma_commit(empty_bar);
                        if (last) umma_commit(bar_accfull + 8 * buf);
                    }
                    __syncwarp();
                    ring.advance(nstg);
                }
                acc_use[buf]++;
                buf ^= 1;
            }
        }
    } else {
        // ---------------- epilogue: thread = token row = TMEM lane; two warps per lane quarter split the channels ----------------
        const int quarter = warp & 3;                      // this warp may touch TMEM lanes 32 * (warp % 4) .. + 31
        const int colhalf = (warp - 2) >> 2;               // which half of an accumulator's channels
        const int row = quarter * 32 + lane;
        const uint32_t cs_base = sbase + L::cs_off;
        DnTile ti;
        bool ok = true;
        uint32_t acc_use[2] = {0, 0};
        int buf = 0, cs_e = -1;
        DnTile nx;
        bool have = dn_tile(s_off, p.E, blockIdx.x, nx);
        long long next_yrow = (have && row < nx.rows) ? p.perm[nx.m0 + row] : 0;     // fetched one tile ahead
        for (int t = blockIdx.x; ok && have; t += gridDim.x) {
            ti = nx;
            const long long yrow = next_yrow;
            have = dn_tile(s_off, p.E, t + gridDim.x, nx);
            next_yrow = (have && row < nx.rows) ? p.perm[nx.m0 + row] : 0;
            if (ti.e != cs_e) {
                // the column scales of this expert, staged once per change of expert by the epilogue warps
                asm volatile("bar.sync 1, %0;" ::"n"(DN_EPI_THREADS) : "memory");
                for (int i = tid - 64; i < p.Np; i += DN_EPI_THREADS) s_cs[i] = p.col_scale[(size_t)ti.e * p.Np + i];
                asm volatile("bar.sync 1, %0;" ::"n"(DN_EPI_THREADS) : "memory");
                cs_e = ti.e;
            }
            const bool live = row < ti.rows;
            const uint32_t out_row = out_base + row * out_pitch;
            for (int nc = 0; ok && nc < nchunks; ++nc) {
                const int wrows = min(DN_NC, p.Nw - nc * DN_NC);
                const int half_cols = wrows >> 1, c_lo = colhalf * half_cols;          // this warp's channels of the chunk
                if (!(ok = mbar_wait(bar_accfull + 8 * buf, acc_use[buf] & 1u, s_abort, p.status))) break;
                tc_fence_after();
                // the previous chunk's row has left shared memory (this thread's own bulk store) before it is overwritten
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                for (int c = c_lo; c < c_lo + half_cols; c += 32) {
                    uint32_t v[32];
                    tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * DN_NC + c, v);
                    tmem_ld_wait();
                    const uint32_t cs = cs_base + (nc * DN_NC + c) * 4;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float sc[8];
                        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(sc[0]), "=f"(sc[1]), "=f"(sc[2]), "=f"(sc[3]) : "r"(cs + j * 32));
                        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(sc[4]), "=f"(sc[5]), "=f"(sc[6]), "=f"(sc[7]) : "r"(cs + j * 32 + 16));
                        uint32_t o[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[8 * j + 2 * i]) * sc[2 * i],
                                                                     __uint_as_float(v[8 * j + 2 * i + 1]) * sc[2 * i + 1]);
                            o[i] = *reinterpret_cast<uint32_t*>(&h);
                        }
                        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(out_row + (c + 8 * j) * 2), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
                    }
                }
                tc_fence_before();
                mbar_arrive(bar_accempty + 8 * buf);
                acc_use[buf]++;
                buf ^= 1;
                // this warp's channels of the row go out as ONE contiguous copy to the row's original position
                const int n0 = nc * DN_NC + c_lo, nbytes = min(half_cols, p.N - n0) * 2;
                if (live && nbytes > 0) {
                    fence_proxy_async();
                    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                                 ::"l"(p.Y + yrow * p.N + n0), "r"(out_row + c_lo * 2), "r"(nbytes) : "memory");
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
        }
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (*s_abort) {
        unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn dn_encode_fn() {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
        return (EncodeTiledFn)f;
    return nullptr;
}
bool dn_map(EncodeTiledFn enc, CUtensorMap* m, const void* base, size_t rows, size_t cols) {
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, 64};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
size_t al256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

// what this kernel takes: a large batch, K at most 1024 (see the header), weights of all
// experts together small enough to stay cache-resident as dense bf16
bool dense_supported(int M, int N, int K, const moqe_expert* const* ex, int E) {
    if (M <= 128 || K % 8 != 0 || K > DN_MAX_K || N % 8 != 0) return false;
    const size_t Np = ex[0]->Np, Kp = ex[0]->Kp;
    return Np <= 1024 && Np * Kp * 4 * (size_t)E <= (size_t)32 << 20;
}

size_t dense_workspace_bytes(int M, int K, int E, int Np, int Kp) {
    (void)M; (void)K;
    return al256((size_t)E * Np * Kp * 4) + al256((size_t)E * Np * 4);
}

moqe_status launch_qgemm_dense(const void* X, int M, int N, int K, const moqe_expert* const* ex, int E, void* Y,
                               const int32_t* perm, const int32_t* offsets, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (M == 0) return MOQE_OK;
    if (!dense_supported(M, N, K, ex, E)) return MOQE_ERR_UNSUPPORTED;
    const int Np = ex[0]->Np, Kp = ex[0]->Kp;
    if (!ws || ws_bytes < dense_workspace_bytes(M, K, E, Np, Kp)) return MOQE_ERR_WORKSPACE;
    EncodeTiledFn enc = dn_encode_fn();
    if (!enc) return MOQE_ERR_CUDA;
    char* base = (char*)ws;
    uint16_t* Wd = (uint16_t*)base;
    float* cs = (float*)(base + al256((size_t)E * Np * Kp * 4));
    moqe_status s = launch_dense_unpack(ex, E, Wd, cs, st);
    if (s != MOQE_OK) return s;
    CUtensorMap tmap_x, tmap_w;
    if (!dn_map(enc, &tmap_x, X, M, K) || !dn_map(enc, &tmap_w, Wd, (size_t)E * Np, 2 * (size_t)Kp))
        return MOQE_ERR_CUDA;
    DnParams p;
    p.perm = perm; p.offsets = offsets; p.X = (const uint16_t*)X; p.col_scale = cs; p.Y = (uint16_t*)Y;
    p.status = device_status_word();
    p.M = M; p.N = N; p.K = K; p.Np = Np; p.Kp = Kp; p.E = E; p.Ksteps = (K + 63) / 64;
    p.Nw = (N + 63) / 64 * 64;
    p.split_mask = 0;
    for (int e = 0; e < E; ++e)
        if (ex[e]->group != 0) p.split_mask |= 1u << e;
    p.max_steps = p.Ksteps * (p.split_mask ? 2 : 1);
    p.resident = (size_t)p.max_steps * p.Nw * 128 <= (size_t)DN_WRES_MAX ? 1 : 0;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long tiles = (long long)(M + 127) / 128 + E;
    const int grid = (int)(tiles < sms ? tiles : sms);
    if (cudaFuncSetAttribute(qgemm_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DnSmem::dyn_bytes) != cudaSuccess)
        return MOQE_ERR_CUDA;
    qgemm_dense_kernel<<<grid, DN_THREADS, DnSmem::dyn_bytes, st>>>(p, tmap_x, tmap_w);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

}  // namespace moqe
