// Routed dequant-GEMM for small batches (decode shapes): every touched expert's
// packed weights are streamed from HBM exactly once with 128-bit loads, unpacked
// in registers to exact small integers (c - z) in bf16, and multiplied against
// the expert's few token rows with warp-level m16n8k16 tensor-core MMAs
// (weights are the 16-row operand, tokens the 8-column operand).  Group scales
// are applied in fp32 outside the MMA ("two-level accumulation"):
//
//   Y[m][n] = sum_groups s[n][G] * ( sum_{k in G} X[m][k] * (c[n][k] - z[n][G]) )
//
// so the tensor core only ever sees exactly representable operands and the
// result differs from an fp32 reference by summation order alone.
//
// Work decomposition: task = (expert, 128-channel tile, K split).  K is split so
// that tasks carry about equal bytes whatever the expert's bit-width.  Split
// partials go to a workspace; the last CTA to arrive for a (tile, token chunk)
// adds them in fixed split order and writes bf16 rows straight to their
// original (unsorted) positions, which fuses the un-permutation.
//
// Section 3.1 of the paper ("the activated quantization expert performs the
// inference on this sample") is the operation; the paper describes no kernel.
#include <type_traits>

#include "dequant.cuh"

namespace moqe {
namespace {

constexpr int STREAM_THREADS = 256;          // 8 warps = the 8 blobs (16 channels each) of a 128-channel tile
constexpr int KC_BLOBS = 8;                  // X is staged in shared memory 8 blobs (1024 k) at a time
constexpr int XS_STRIDE = KC_BLOBS * 128 * 2 + 64;   // bytes per staged token row; = 64 mod 128: conflict-free LDS.128
constexpr int OUT_STRIDE = 132;              // floats per staged output row
constexpr int SPLIT_MAX_ROWS = 64;           // K is split only for batches this small (partials: MAX_SPLIT*M*Np floats)
constexpr int MAX_SPLIT = 16;

struct StreamParams {
    ExpertDev ex[MOQE_MAX_EXPERTS];
    int task_base[MOQE_MAX_EXPERTS + 1];
    int ksplit[MOQE_MAX_EXPERTS];
    const uint16_t* X;
    uint16_t* Y;
    const int32_t* perm;
    const int32_t* offsets;
    float* partials;        // [split][M][Np]
    uint32_t* counters;     // [ntiles][M]
    int* status;
    int M, N, K, Np, KB, E, ntiles;
};

__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ldg_stream8(const void* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// The raw packed words one lane holds for one blob: the pieces of channel rows
// gl (lo) and gl + 8 (hi), gl = lane / 4, at k quarter q = lane % 4.
template <int BITS>
struct LaneBlob { uint32_t lo[PieceWords<BITS>::n], hi[PieceWords<BITS>::n]; };

template <int BITS>
__device__ __forceinline__ void load_blob(LaneBlob<BITS>& b, const uint8_t* blob, int slot) {
    if constexpr (BITS == 4) {
        uint4 l = ldg_stream16(blob + slot * 16), h = ldg_stream16(blob + 512 + slot * 16);
        b.lo[0] = l.x; b.lo[1] = l.y; b.lo[2] = l.z; b.lo[3] = l.w;
        b.hi[0] = h.x; b.hi[1] = h.y; b.hi[2] = h.z; b.hi[3] = h.w;
    } else if constexpr (BITS == 8) {
        uint4 l0 = ldg_stream16(blob + slot * 16), l1 = ldg_stream16(blob + 512 + slot * 16);
        uint4 h0 = ldg_stream16(blob + 1024 + slot * 16), h1 = ldg_stream16(blob + 1536 + slot * 16);
        b.lo[0] = l0.x; b.lo[1] = l0.y; b.lo[2] = l0.z; b.lo[3] = l0.w;
        b.lo[4] = l1.x; b.lo[5] = l1.y; b.lo[6] = l1.z; b.lo[7] = l1.w;
        b.hi[0] = h0.x; b.hi[1] = h0.y; b.hi[2] = h0.z; b.hi[3] = h0.w;
        b.hi[4] = h1.x; b.hi[5] = h1.y; b.hi[6] = h1.z; b.hi[7] = h1.w;
    } else {
        uint4 x = ldg_stream16(blob + slot * 16);
        uint2 y = ldg_stream8(blob + 512 + slot * 8);
        b.lo[0] = x.x; b.lo[1] = x.y; b.lo[2] = x.z;
        b.hi[0] = x.w; b.hi[1] = y.x; b.hi[2] = y.y;
    }
}

__device__ __forceinline__ float pick4(const float (&a)[4], int j) { return j == 0 ? a[0] : j == 1 ? a[1] : j == 2 ? a[2] : a[3]; }

// per-blob scale / zero-point values of the lane's two channel rows (up to 4 groups per blob)
struct BlobMeta { float s_lo[4], s_hi[4], z_lo[4], z_hi[4]; };

__device__ __forceinline__ void load_meta(BlobMeta& m, const ExpertDev& ex, int Np, int kb, int n_lo, int ngrp, int sym_z) {
    // ngrp = groups per blob (1, 2 or 4); group index of sub-group j: kb*ngrp + j  (group >= 128: (kb*128)/group)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (j < ngrp) {
            size_t gi = (ex.group >= 128) ? (size_t)(kb * 128 / ex.group) : (size_t)(kb * ngrp + j);
            const __half* sp = ex.scales_t + gi * Np + n_lo;
            m.s_lo[j] = __half2float(sp[0]);
            m.s_hi[j] = __half2float(sp[8]);
            if (ex.zeros_t) {
                const __nv_bfloat16* zp = ex.zeros_t + gi * Np + n_lo;
                m.z_lo[j] = __bfloat162float(zp[0]);
                m.z_hi[j] = __bfloat162float(zp[8]);
            } else {
                m.z_lo[j] = m.z_hi[j] = (float)sym_z;
            }
        }
    }
}

template <int BITS, int NT>
__device__ __forceinline__ void run_task(const StreamParams& p, const ExpertDev& ex, int nt, int split, int S, int row0,
                                         int rows, unsigned char* smem) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gl = lane >> 2, q = lane & 3;
    const int slot = q * 8 + gl;
    constexpr int T = 8 * NT;
    const int kb0 = (int)((long long)split * p.KB / S), kb1 = (int)((long long)(split + 1) * p.KB / S);
    const int n_lo = nt * 128 + warp * 16 + gl;                     // this lane's first channel row (second: +8)
    const int sym_z = 1 << (BITS - 1);
    const bool per_channel = ex.group == 0;
    const int ngrp = per_channel ? 1 : (ex.group >= 128 ? 1 : 128 / ex.group);
    const size_t blob_bytes = (size_t)moqe_blob_bytes(BITS);
    const uint8_t* blob_base = ex.codes + ((size_t)nt * p.KB * 8 + warp) * blob_bytes;   // + kb * 8 * blob_bytes
    float* out = reinterpret_cast<float*>(smem);
    __shared__ int s_last;

    for (int c0 = 0; c0 < rows; c0 += T) {
        const int tvalid = min(T, rows - c0);
        float acc[NT][4], part[NT][4];
#pragma unroll
        for (int i = 0; i < NT; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = part[i][j] = 0.f;

        LaneBlob<BITS> cur, nxt;
        BlobMeta mcur, mnxt;
        if (kb0 < kb1) {
            load_blob<BITS>(cur, blob_base + (size_t)kb0 * 8 * blob_bytes, slot);
            if (per_channel) load_meta(mcur, ex, p.Np, 0, n_lo, 1, sym_z);
            else load_meta(mcur, ex, p.Np, kb0, n_lo, ngrp, sym_z);
        }
        for (int kc0 = kb0; kc0 < kb1; kc0 += KC_BLOBS) {
            const int nblob = min(KC_BLOBS, kb1 - kc0);
            __syncthreads();                                        // previous stage (or output staging) consumed
            // stage X[perm[row0 + c0 + tok]][kc0*128 .. ) : 16 bytes per thread per step, zero beyond rows / K
            const int vec_per_row = nblob * 16;
            for (int i = tid; i < T * vec_per_row; i += STREAM_THREADS) {
                int tok = i / vec_per_row, v = i - tok * vec_per_row;
                int k = kc0 * 128 + v * 8;
                uint4 val = make_uint4(0, 0, 0, 0);
                if (tok < tvalid && k < p.K) {
                    int src = p.perm[row0 + c0 + tok];
                    val = *reinterpret_cast<const uint4*>(p.X + (size_t)src * p.K + k);
                }
                *reinterpret_cast<uint4*>(smem + tok * XS_STRIDE + v * 16) = val;
            }
            __syncthreads();
            for (int kb = kc0; kb < kc0 + nblob; ++kb) {
                if (kb + 1 < kb1) {
                    load_blob<BITS>(nxt, blob_base + (size_t)(kb + 1) * 8 * blob_bytes, slot);
                    if (!per_channel) load_meta(mnxt, ex, p.Np, kb + 1, n_lo, ngrp, sym_z);
                }
                const unsigned char* xrow = smem + gl * XS_STRIDE + ((kb - kc0) * 128 + 8 * q) * 2;
                auto chunk = [&](auto Gc) {
                    constexpr int G = decltype(Gc)::value;
                    const int gj = per_channel ? 0 : (ngrp == 4 ? G : (ngrp == 2 ? (G >> 1) : 0));
                    uint32_t lo[4], hi[4];
                    unpack_chunk<BITS, G>(cur.lo, pick4(mcur.z_lo, gj), lo);
                    unpack_chunk<BITS, G>(cur.hi, pick4(mcur.z_hi, gj), hi);
#pragma unroll
                    for (int t = 0; t < NT; ++t) {
                        uint4 xb = *reinterpret_cast<const uint4*>(xrow + t * 8 * XS_STRIDE + G * 64);
                        mma_bf16(part[t], lo[0], hi[0], lo[1], hi[1], xb.x, xb.y);
                        mma_bf16(part[t], lo[2], hi[2], lo[3], hi[3], xb.z, xb.w);
                    }
                    const bool promote = !per_channel && (ngrp == 4 || (ngrp == 2 && (G & 1)) || (ngrp == 1 && G == 3));
                    if (promote) {
                        const float sl = pick4(mcur.s_lo, gj), sh = pick4(mcur.s_hi, gj);
#pragma unroll
                        for (int t = 0; t < NT; ++t) {
                            acc[t][0] = fmaf(sl, part[t][0], acc[t][0]);
                            acc[t][1] = fmaf(sl, part[t][1], acc[t][1]);
                            acc[t][2] = fmaf(sh, part[t][2], acc[t][2]);
                            acc[t][3] = fmaf(sh, part[t][3], acc[t][3]);
                            part[t][0] = part[t][1] = part[t][2] = part[t][3] = 0.f;
                        }
                    }
                };
                chunk(std::integral_constant<int, 0>{});
                chunk(std::integral_constant<int, 1>{});
                chunk(std::integral_constant<int, 2>{});
                chunk(std::integral_constant<int, 3>{});
                if (kb + 1 < kb1) {
                    cur = nxt;
                    if (!per_channel) mcur = mnxt;
                }
            }
        }
        if (per_channel && kb0 < kb1) {
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                acc[t][0] = mcur.s_lo[0] * part[t][0];
                acc[t][1] = mcur.s_lo[0] * part[t][1];
                acc[t][2] = mcur.s_hi[0] * part[t][2];
                acc[t][3] = mcur.s_hi[0] * part[t][3];
            }
        }
        // ---- stage the [T][128] fp32 tile through shared memory -------------------------------
        __syncthreads();                                            // X stage no longer needed
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            int tok = t * 8 + 2 * q, nl = warp * 16 + gl;
            out[tok * OUT_STRIDE + nl] = acc[t][0];
            out[(tok + 1) * OUT_STRIDE + nl] = acc[t][1];
            out[tok * OUT_STRIDE + nl + 8] = acc[t][2];
            out[(tok + 1) * OUT_STRIDE + nl + 8] = acc[t][3];
        }
        __syncthreads();
        const int j0 = row0 + c0;
        bool write_final = true;
        if (S > 1) {
            for (int i = tid; i < tvalid * 32; i += STREAM_THREADS) {
                int tok = i >> 5, v = i & 31;
                float4 val = *reinterpret_cast<const float4*>(out + tok * OUT_STRIDE + v * 4);
                *reinterpret_cast<float4*>(p.partials + ((size_t)split * p.M + j0 + tok) * p.Np + nt * 128 + v * 4) = val;
            }
            __threadfence();
            __syncthreads();
            if (tid == 0) {
                unsigned* cnt = p.counters + (size_t)nt * p.M + j0;
                unsigned old = atomicAdd(cnt, 1u);
                s_last = (old == (unsigned)(S - 1));
                if (s_last) *cnt = 0u;                              // leave the counters clear for the next call
            }
            __syncthreads();
            write_final = s_last != 0;
            if (write_final) __threadfence();
        }
        if (write_final) {
            for (int i = tid; i < tvalid * 64; i += STREAM_THREADS) {
                int tok = i >> 6, v = i & 63;
                int n = nt * 128 + v * 2;
                if (n >= p.N) continue;                             // N is even
                float a, b;
                if (S > 1) {
                    a = b = 0.f;
                    for (int s2 = 0; s2 < S; ++s2) {
                        float2 pv = __ldcg(reinterpret_cast<const float2*>(p.partials + ((size_t)s2 * p.M + j0 + tok) * p.Np + n));
                        a += pv.x;
                        b += pv.y;
                    }
                } else {
                    a = out[tok * OUT_STRIDE + v * 2];
                    b = out[tok * OUT_STRIDE + v * 2 + 1];
                }
                int dst = p.perm[j0 + tok];
                *reinterpret_cast<uint32_t*>(p.Y + (size_t)dst * p.N + n) = pack_bf16x2(a, b);
            }
        }
    }
}

template <int NT>
__global__ void __launch_bounds__(STREAM_THREADS, 2) qgemm_stream_kernel(const __grid_constant__ StreamParams p) {
    extern __shared__ __align__(16) unsigned char smem[];
    int task = blockIdx.x;
    int e = 0;
    while (e + 1 < p.E && task >= p.task_base[e + 1]) ++e;
    const int local = task - p.task_base[e];
    const int S = p.ksplit[e];
    const int nt = local / S, split = local - nt * S;
    const int row0 = p.offsets[e];
    const int rows = p.offsets[e + 1] - row0;
    if (rows <= 0) return;
    const ExpertDev& ex = p.ex[e];
    if (ex.bits == 4) run_task<4, NT>(p, ex, nt, split, S, row0, rows, smem);
    else if (ex.bits == 8) run_task<8, NT>(p, ex, nt, split, S, row0, rows, smem);
    else run_task<3, NT>(p, ex, nt, split, S, row0, rows, smem);
}

template <int NT>
size_t stream_smem_bytes() {
    size_t x = (size_t)8 * NT * XS_STRIDE, o = (size_t)8 * NT * OUT_STRIDE * 4;
    return x > o ? x : o;
}

int pick_nt(int M) { return M <= 8 ? 1 : (M <= 16 ? 2 : 4); }

// K splits per expert: tasks of about equal bytes, enough of them to fill the machine a few times over
void plan_splits(const moqe_expert* const* ex, int E, int M, int sm_count, int* ksplit, int* max_split) {
    const int KB = ex[0]->Kp / 128, ntiles = ex[0]->Np / 128;
    size_t total = 0;
    for (int e = 0; e < E; ++e) total += (size_t)ex[e]->Np * ex[e]->Kp * ex[e]->bits / 8;
    size_t target = total / ((size_t)sm_count * 2 * 3);
    if (target < 32 * 1024) target = 32 * 1024;
    *max_split = 1;
    for (int e = 0; e < E; ++e) {
        size_t tile_bytes = (size_t)128 * ex[e]->Kp * ex[e]->bits / 8;
        int s = (int)((tile_bytes + target / 2) / target);
        if (s < 1) s = 1;
        if (s > KB) s = KB;
        if (s > MAX_SPLIT) s = MAX_SPLIT;
        if (M > SPLIT_MAX_ROWS) s = 1;              // split partials are only worth it for small batches
        ksplit[e] = s;
        if (s > *max_split) *max_split = s;
    }
    (void)ntiles;
}

int g_sm_count = 0;
int sm_count() {
    if (!g_sm_count) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (g_sm_count <= 0) g_sm_count = 148;
    }
    return g_sm_count;
}

}  // namespace

size_t stream_zero_bytes(int M, int Np) { return M > SPLIT_MAX_ROWS ? 0 : (size_t)(Np / 128) * M * sizeof(uint32_t); }

size_t stream_workspace_bytes(int M, int Np, int E) {
    (void)E;
    if (M > SPLIT_MAX_ROWS) return 0;
    size_t counters = (stream_zero_bytes(M, Np) + 255) / 256 * 256;
    size_t partials = (size_t)MAX_SPLIT * M * Np * sizeof(float);
    return counters + partials;
}

moqe_status launch_qgemm_stream(const void* X, int M, int N, int K, const moqe_expert* const* ex, int E, void* Y,
                                const int32_t* perm, const int32_t* offsets, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (M == 0) return MOQE_OK;
    StreamParams p;
    int max_split = 1;
    plan_splits(ex, E, M, sm_count(), p.ksplit, &max_split);
    p.KB = ex[0]->Kp / 128;
    p.Np = ex[0]->Np;
    p.ntiles = p.Np / 128;
    int tasks = 0;
    for (int e = 0; e < E; ++e) {
        p.ex[e].codes = ex[e]->codes;
        p.ex[e].scales_t = ex[e]->scales_t;
        p.ex[e].zeros_t = ex[e]->zeros_t;
        p.ex[e].bits = ex[e]->bits;
        p.ex[e].group = ex[e]->group;
        p.task_base[e] = tasks;
        tasks += p.ntiles * p.ksplit[e];
    }
    p.task_base[E] = tasks;
    p.X = (const uint16_t*)X;
    p.Y = (uint16_t*)Y;
    p.perm = perm;
    p.offsets = offsets;
    p.M = M; p.N = N; p.K = K; p.E = E;
    p.status = device_status_word();
    p.counters = nullptr;
    p.partials = nullptr;
    if (max_split > 1) {
        if (!ws || ws_bytes < stream_workspace_bytes(M, p.Np, E)) return MOQE_ERR_WORKSPACE;
        p.counters = (uint32_t*)ws;
        p.partials = (float*)((char*)ws + (stream_zero_bytes(M, p.Np) + 255) / 256 * 256);
    }
    const int nt = pick_nt(M);
    cudaError_t err = cudaSuccess;
#define MOQE_LAUNCH(NT)                                                                                           \
    do {                                                                                                          \
        static bool attr_set = false;                                                                             \
        size_t smem = stream_smem_bytes<NT>();                                                                    \
        if (!attr_set) {                                                                                          \
            err = cudaFuncSetAttribute(qgemm_stream_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
            attr_set = (err == cudaSuccess);                                                                      \
        }                                                                                                         \
        if (err == cudaSuccess) qgemm_stream_kernel<NT><<<tasks, STREAM_THREADS, smem, st>>>(p);                  \
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
