// Hard routing (arg-max), stable counting sort of rows by expert id, and the
// row gather / scatter around the grouped GEMM.
//
// Section 3.2 / Appendix of the paper: the router's decision is one expert
// index per sample.  The sort is the batching glue that turns "one expert per
// sample" into contiguous per-expert row segments; its per-expert counts are
// the n_i of the load statistic F_i = n_i / B (Section 3.3).
//
// Sort: bucket = id for valid ids, bucket E for ids outside [0,E) (those rows
// end up behind all valid rows and latch MOQE_ERR_EXPERT_ID).  Within a warp
// the stable rank of a row among equal ids comes from __match_any_sync; warps
// and blocks are combined with prefix sums, so perm is the unique stable order.
#include <mutex>

#include "common.cuh"

namespace moqe {
namespace {

constexpr int SORT_THREADS = 1024;
constexpr int SORT_WARPS = SORT_THREADS / 32;
constexpr int MAXB = MOQE_MAX_EXPERTS + 1;   // buckets incl. the invalid-id bucket

// first maximum of one row of logits; NaN never wins; a row of NaNs gives 0
__device__ __forceinline__ int first_argmax(const float* __restrict__ l, int E) {
    int best = -1;
    float bv = 0.f;
    for (int e = 0; e < E; ++e) {
        float v = l[e];
        if (v != v) continue;
        if (best < 0 || v > bv) { best = e; bv = v; }
    }
    return best < 0 ? 0 : best;
}

__global__ void route_kernel(const float* __restrict__ logits, int S, int E, int32_t* __restrict__ ids) {
    int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= S) return;
    ids[s] = first_argmax(logits + (size_t)s * E, E);
}

__global__ void expand_ids_kernel(const int32_t* __restrict__ ids, const int32_t* __restrict__ row_offsets, int S, int M,
                                  int32_t* __restrict__ row_ids) {
    int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= M) return;
    // largest s with row_offsets[s] <= m  (row_offsets is non-decreasing, row_offsets[0] = 0)
    int lo = 0, hi = S;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (row_offsets[mid] <= m) lo = mid; else hi = mid;
    }
    row_ids[m] = ids[lo];
}

// Per-block pieces of the sort --------------------------------------------------
// Stable rank of each of this block's rows inside the block, and per-bucket block
// totals.  Row m = base + threadIdx.x.  On return (after the trailing barrier)
// s_warp[w][b] = number of rows of bucket b in warps < w of this block, and
// s_tot[b] = rows of bucket b in the block.
struct BlockRank { int bucket; int rank; bool live; };

__device__ __forceinline__ BlockRank block_rank(const int32_t* __restrict__ row_ids, int M, int E, long long base,
                                                int (*s_warp)[MAXB], int* s_tot, int* status) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    long long m = base + threadIdx.x;
    BlockRank br;
    br.live = m < M;
    int id = br.live ? row_ids[m] : 0;
    bool bad = br.live && (id < 0 || id >= E);
    if (bad) latch_status(status, (int)MOQE_ERR_EXPERT_ID);
    br.bucket = bad ? E : id;
    for (int i = threadIdx.x; i < SORT_WARPS * MAXB; i += blockDim.x) (&s_warp[0][0])[i] = 0;
    __syncthreads();
    unsigned live_mask = __ballot_sync(0xffffffffu, br.live);
    int rank_in_warp = 0;
    if (br.live) {
        unsigned peers = __match_any_sync(live_mask, br.bucket);
        rank_in_warp = __popc(peers & ((1u << lane) - 1u));
        if (rank_in_warp == 0) s_warp[warp][br.bucket] = __popc(peers);
    }
    __syncthreads();
    if (threadIdx.x <= E) {                         // exclusive scan over warps, one thread per bucket
        int run = 0;
        for (int w = 0; w < SORT_WARPS; ++w) { int c = s_warp[w][threadIdx.x]; s_warp[w][threadIdx.x] = run; run += c; }
        s_tot[threadIdx.x] = run;
    }
    __syncthreads();
    br.rank = rank_in_warp + (br.live ? s_warp[warp][br.bucket] : 0);
    return br;
}

__device__ __forceinline__ void zero_row(void* Y, int N, long long row) {
    // one thread zeroes a whole row: only rows with an invalid id take this path
    uint4* y = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(Y) + (size_t)row * N);
    for (int i = 0; i < N / 8; ++i) y[i] = make_uint4(0, 0, 0, 0);
}

// M <= 1024: the whole sort in one block; also clears `zero_region` (split-K arrival counters).
__global__ void __launch_bounds__(SORT_THREADS) sort_small_kernel(const int32_t* __restrict__ row_ids, int M, int E,
                                                                  int32_t* __restrict__ perm, int32_t* __restrict__ offsets,
                                                                  uint32_t* __restrict__ zero_region, size_t zero_words,
                                                                  void* Y, int N, int* status) {
    __shared__ int s_warp[SORT_WARPS][MAXB];
    __shared__ int s_tot[MAXB];
    __shared__ int s_off[MAXB + 1];
    for (size_t i = threadIdx.x; i < zero_words; i += blockDim.x) zero_region[i] = 0u;
    BlockRank br = block_rank(row_ids, M, E, 0, s_warp, s_tot, status);
    if (threadIdx.x == 0) {
        int run = 0;
        for (int b = 0; b <= E; ++b) { s_off[b] = run; run += s_tot[b]; }
        s_off[E + 1] = run;
    }
    __syncthreads();
    if (threadIdx.x <= E) offsets[threadIdx.x] = s_off[threadIdx.x];
    if (br.live) {
        perm[s_off[br.bucket] + br.rank] = threadIdx.x;
        if (br.bucket == E && Y) zero_row(Y, N, threadIdx.x);
    }
}

// Route, expand and sort in one block for a batch of at most 1024 rows and 1024 samples: thread s < S takes the arg-max
// of sample s, thread m < M looks up its sample and sorts as sort_small_kernel does.  Dependents may be scheduled at
// once (they wait for this grid's results themselves).
__global__ void __launch_bounds__(SORT_THREADS) route_sort_small_kernel(const float* __restrict__ logits, int S, int E,
                                                                        const int32_t* __restrict__ row_offsets, int M,
                                                                        int32_t* __restrict__ ids, int32_t* __restrict__ row_ids,
                                                                        int32_t* __restrict__ perm, int32_t* __restrict__ offsets) {
    __shared__ int s_warp[SORT_WARPS][MAXB];
    __shared__ int s_tot[MAXB];
    __shared__ int s_off[MAXB + 1];
    __shared__ int s_ids[SORT_THREADS];
    __shared__ int s_rows[SORT_THREADS];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int t = threadIdx.x;
    if (t < S) {
        const int id = first_argmax(logits + (size_t)t * E, E);
        s_ids[t] = id;
        ids[t] = id;
    }
    if (t < S) s_rows[t] = row_offsets ? row_offsets[t] : t;
    __syncthreads();
    const int lane = t & 31, warp = t >> 5;
    const bool live = t < M;
    int bucket = 0;
    if (live) {
        int lo = 0, hi = S;                          // largest s with row_offsets[s] <= m
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (s_rows[mid] <= t) lo = mid; else hi = mid;
        }
        bucket = s_ids[lo];                          // valid by construction
        row_ids[t] = bucket;
    }
    for (int i = t; i < SORT_WARPS * MAXB; i += blockDim.x) (&s_warp[0][0])[i] = 0;
    __syncthreads();
    const unsigned live_mask = __ballot_sync(0xffffffffu, live);
    int rank_in_warp = 0;
    if (live) {
        const unsigned peers = __match_any_sync(live_mask, bucket);
        rank_in_warp = __popc(peers & ((1u << lane) - 1u));
        if (rank_in_warp == 0) s_warp[warp][bucket] = __popc(peers);
    }
    __syncthreads();
    if (t <= E) {
        int run = 0;
        for (int w = 0; w < SORT_WARPS; ++w) { int c = s_warp[w][t]; s_warp[w][t] = run; run += c; }
        s_tot[t] = run;
    }
    __syncthreads();
    if (t == 0) {
        int run = 0;
        for (int b = 0; b <= E; ++b) { s_off[b] = run; run += s_tot[b]; }
        s_off[E + 1] = run;
    }
    __syncthreads();
    if (t <= E) offsets[t] = s_off[t];
    if (live) perm[s_off[bucket] + rank_in_warp + s_warp[warp][bucket]] = t;
}

// M > 1024: three kernels.  (1) per-block bucket totals
__global__ void __launch_bounds__(SORT_THREADS) sort_hist_kernel(const int32_t* __restrict__ row_ids, int M, int E,
                                                                 int32_t* __restrict__ block_tot, int* status) {
    __shared__ int s_warp[SORT_WARPS][MAXB];
    __shared__ int s_tot[MAXB];
    block_rank(row_ids, M, E, (long long)blockIdx.x * SORT_THREADS, s_warp, s_tot, status);
    if (threadIdx.x <= E) block_tot[(size_t)blockIdx.x * MAXB + threadIdx.x] = s_tot[threadIdx.x];
}

// (2) exclusive scan in (bucket-major, block-minor) order; block_tot becomes the base slot of (block, bucket).
// One warp per bucket: the lanes read 32 consecutive blocks' totals, scan them with shuffles and carry the running
// sum to the next 32 (a serial walk over all blocks costs two dependent global round trips per block).
__global__ void __launch_bounds__(1024) sort_scan_kernel(int32_t* __restrict__ block_tot, int nblk, int E,
                                                              int32_t* __restrict__ offsets) {
    __shared__ int s_sum[MAXB];
    __shared__ int s_off[MAXB + 1];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int b = warp; b <= E; b += 32) {
        int run = 0;
        for (int i0 = 0; i0 < nblk; i0 += 32) {
            const int i = i0 + lane;
            const int c = i < nblk ? block_tot[(size_t)i * MAXB + b] : 0;
            int incl = c;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += o;
            }
            if (i < nblk) block_tot[(size_t)i * MAXB + b] = run + incl - c;
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) s_sum[b] = run;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int i = 0; i <= E; ++i) { s_off[i] = run; run += s_sum[i]; }
    }
    __syncthreads();
    for (int b = warp; b <= E; b += 32) {
        const int off = s_off[b];
        if (lane == 0) offsets[b] = off;
        for (int i = lane; i < nblk; i += 32) block_tot[(size_t)i * MAXB + b] += off;
    }
}

// (3) scatter row indices to their slots
__global__ void __launch_bounds__(SORT_THREADS) sort_scatter_kernel(const int32_t* __restrict__ row_ids, int M, int E,
                                                                    const int32_t* __restrict__ block_base,
                                                                    int32_t* __restrict__ perm, void* Y, int N) {
    __shared__ int s_warp[SORT_WARPS][MAXB];
    __shared__ int s_tot[MAXB];
    long long base = (long long)blockIdx.x * SORT_THREADS;
    BlockRank br = block_rank(row_ids, M, E, base, s_warp, s_tot, nullptr);
    if (br.live) {
        long long m = base + threadIdx.x;
        perm[block_base[(size_t)blockIdx.x * MAXB + br.bucket] + br.rank] = (int32_t)m;
        if (br.bucket == E && Y) zero_row(Y, N, m);
    }
}

// Row gather / scatter: 16 bytes per thread, a row is covered by consecutive threads.
// GATHER : dst[j] = src[perm[j]]   (rows j >= n_valid, i.e. invalid ids, are zero-filled)
// SCATTER: dst[perm[j]] = src[j]
template <bool GATHER>
__global__ void move_rows_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ perm,
                                 const int32_t* __restrict__ n_valid_ptr, long long M, int vec_per_row,
                                 uint4* __restrict__ dst) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M * vec_per_row) return;
    long long j = i / vec_per_row;
    int v = (int)(i % vec_per_row);
    long long p = perm[j];
    if (GATHER) {
        bool valid = !n_valid_ptr || j < *n_valid_ptr;
        dst[j * vec_per_row + v] = valid ? src[p * vec_per_row + v] : make_uint4(0, 0, 0, 0);
    } else {
        dst[p * vec_per_row + v] = src[j * vec_per_row + v];
    }
}

// Gather for the tcgen05 kernel, 64-row box by box.  Boxes are counted per expert from the start of the
// expert's segment (box id = sum over earlier experts of ceil(rows/64) + local box).  A box whose rows are
// consecutive rows of X anyway (the usual case: a sample's rows are contiguous and share an expert) is NOT
// copied: box_src[id] = its first source row, and the GEMM's TMA reads X directly; otherwise the rows are
// copied to Xp[offsets[e] + 64*box ..] and box_src[id] = -1.
// (wide rows: one block per box, so that a box that has to be copied has 256 threads and the grid many blocks)
__global__ void __launch_bounds__(256) gather_boxes_wide_kernel(const uint4* __restrict__ X, const int32_t* __restrict__ perm,
                                                                const int32_t* __restrict__ offsets, int E, int vec_per_row,
                                                                uint4* __restrict__ Xp, int32_t* __restrict__ box_src) {
    int b = blockIdx.x, e = 0, rows_e = 0;
    for (; e < E; ++e) {
        rows_e = offsets[e + 1] - offsets[e];
        const int nb = (rows_e + 63) >> 6;
        if (b < nb) break;
        b -= nb;
    }
    if (e == E) return;
    const int j0 = offsets[e] + b * 64, cnt = min(64, rows_e - b * 64);
    const int first = perm[j0];
    const int ok = (threadIdx.x >= cnt) || (perm[j0 + threadIdx.x] == first + (int)threadIdx.x);
    const int all_ok = __syncthreads_and(ok);
    if (threadIdx.x == 0) box_src[blockIdx.x] = all_ok ? first : -1;
    if (all_ok) return;
    for (int i = threadIdx.x; i < cnt * vec_per_row; i += blockDim.x) {
        const int r = i / vec_per_row, v = i - r * vec_per_row;
        Xp[(size_t)(j0 + r) * vec_per_row + v] = X[(size_t)perm[j0 + r] * vec_per_row + v];
    }
}

// (narrow rows, many boxes: eight boxes per block)
__global__ void __launch_bounds__(256) gather_boxes_kernel(const uint4* __restrict__ X, const int32_t* __restrict__ perm,
                                                           const int32_t* __restrict__ offsets, int E, int vec_per_row,
                                                           uint4* __restrict__ Xp, int32_t* __restrict__ box_src, int nboxes) {
    // one warp per box looks at its 64 rows (lanes: rows l and l + 32); the boxes of the block that have to be
    // copied are then copied by the whole block
    __shared__ int s_j0[8], s_cnt[8];
    const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int box = blockIdx.x * 8 + wib;
    int j0 = 0, cnt = 0;
    if (box < nboxes) {
        int b = box, e = 0, rows_e = 0;
        for (; e < E; ++e) {
            rows_e = offsets[e + 1] - offsets[e];
            const int nb = (rows_e + 63) >> 6;
            if (b < nb) break;
            b -= nb;
        }
        if (e < E) {
            j0 = offsets[e] + b * 64;
            cnt = min(64, rows_e - b * 64);
            const int first = perm[j0];
            const bool ok = (lane >= cnt || perm[j0 + lane] == first + lane) && (lane + 32 >= cnt || perm[j0 + lane + 32] == first + lane + 32);
            const bool all_ok = __all_sync(0xffffffffu, ok);
            if (lane == 0) box_src[box] = all_ok ? first : -1;
            if (all_ok) cnt = 0;
        }
    }
    if (lane == 0) { s_j0[wib] = j0; s_cnt[wib] = cnt; }
    __syncthreads();
    for (int w = 0; w < 8; ++w) {
        const int c = s_cnt[w], base = s_j0[w];
        for (int i = threadIdx.x; i < c * vec_per_row; i += blockDim.x) {
            const int r = i / vec_per_row, v = i - r * vec_per_row;
            Xp[(size_t)(base + r) * vec_per_row + v] = X[(size_t)perm[base + r] * vec_per_row + v];
        }
    }
}

}  // namespace

size_t sort_workspace_bytes(int M, int E) {
    (void)E;
    if (M <= SORT_THREADS) return 256;
    size_t nblk = ((size_t)M + SORT_THREADS - 1) / SORT_THREADS;
    return (nblk * MAXB * sizeof(int32_t) + 255) / 256 * 256;
}

// Sort rows by id.  zero_region (optional, 4-byte multiple) is cleared on the way;
// Y (optional) gets zero rows where the id is invalid.
moqe_status launch_sort(const int32_t* row_ids, int M, int E, int32_t* perm, int32_t* offsets, void* ws, size_t ws_bytes,
                        void* zero_region, size_t zero_bytes, void* Y_zero_invalid, int N, cudaStream_t st) {
    int* status = device_status_word();
    if (!status) return MOQE_ERR_ALLOC;
    if (M <= SORT_THREADS) {
        sort_small_kernel<<<1, SORT_THREADS, 0, st>>>(row_ids, M, E, perm, offsets, (uint32_t*)zero_region,
                                                      zero_bytes / 4, Y_zero_invalid, N, status);
        count_launch();
        return cuda_ok(cudaGetLastError());
    }
    if (!ws || ws_bytes < sort_workspace_bytes(M, E)) return MOQE_ERR_WORKSPACE;
    if (zero_region && zero_bytes) {
        if (cudaMemsetAsync(zero_region, 0, zero_bytes, st) != cudaSuccess) return MOQE_ERR_CUDA;
    }
    int nblk = (M + SORT_THREADS - 1) / SORT_THREADS;
    int32_t* block_tot = (int32_t*)ws;
    sort_hist_kernel<<<nblk, SORT_THREADS, 0, st>>>(row_ids, M, E, block_tot, status);
    sort_scan_kernel<<<1, 1024, 0, st>>>(block_tot, nblk, E, offsets);
    sort_scatter_kernel<<<nblk, SORT_THREADS, 0, st>>>(row_ids, M, E, block_tot, perm, Y_zero_invalid, N);
    count_launch(3);
    return cuda_ok(cudaGetLastError());
}

moqe_status launch_gather(const void* X, const int32_t* perm, const int32_t* n_valid_ptr, int M, int C, void* Xp,
                          cudaStream_t st) {
    if (M == 0) return MOQE_OK;
    int vec = C / 8;
    long long total = (long long)M * vec;
    move_rows_kernel<true><<<(unsigned)((total + 255) / 256), 256, 0, st>>>((const uint4*)X, perm, n_valid_ptr, M, vec,
                                                                           (uint4*)Xp);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

size_t gather_boxes_bytes(int M, int E) { return ((size_t)(M / 64 + E + 1) * sizeof(int32_t) + 255) / 256 * 256; }

moqe_status launch_gather_boxes(const void* X, const int32_t* perm, const int32_t* offsets, int M, int C, int E, void* Xp,
                                int32_t* box_src, cudaStream_t st) {
    if (M == 0) return MOQE_OK;
    const int nboxes = M / 64 + E;
    if (C >= 512 || nboxes < 2048)
        gather_boxes_wide_kernel<<<nboxes, 256, 0, st>>>((const uint4*)X, perm, offsets, E, C / 8, (uint4*)Xp, box_src);
    else
        gather_boxes_kernel<<<(nboxes + 7) / 8, 256, 0, st>>>((const uint4*)X, perm, offsets, E, C / 8, (uint4*)Xp, box_src, nboxes);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

}  // namespace moqe

using namespace moqe;

extern "C" moqe_status moqe_route(const float* logits, int S, int E, int32_t* ids, void* stream) {
    if (!logits || !ids) return MOQE_ERR_NULL;
    if (S < 0 || E <= 0) return MOQE_ERR_SHAPE;
    if (S == 0) return MOQE_OK;
    route_kernel<<<(S + 255) / 256, 256, 0, (cudaStream_t)stream>>>(logits, S, E, ids);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

extern "C" moqe_status moqe_expand_ids(const int32_t* ids, const int32_t* row_offsets, int S, int M, int32_t* row_ids,
                                       void* stream) {
    if (!ids || !row_offsets || !row_ids) return MOQE_ERR_NULL;
    if (S < 0 || M < 0 || (S == 0 && M != 0)) return MOQE_ERR_SHAPE;
    if (M == 0) return MOQE_OK;
    expand_ids_kernel<<<(M + 255) / 256, 256, 0, (cudaStream_t)stream>>>(ids, row_offsets, S, M, row_ids);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

extern "C" moqe_status moqe_route_permute(const float* logits, int S, int E, const int32_t* row_offsets, int M, int32_t* ids,
                                          int32_t* row_ids, int32_t* perm, int32_t* offsets, void* stream) {
    if (!offsets) return MOQE_ERR_NULL;
    if (S < 0 || M < 0 || E <= 0 || (S == 0 && M != 0)) return MOQE_ERR_SHAPE;
    if (!row_offsets && M != S) return MOQE_ERR_SHAPE;
    if (E > MOQE_MAX_EXPERTS || S > SORT_THREADS || M > SORT_THREADS) return MOQE_ERR_UNSUPPORTED;
    if (S > 0 && (!logits || !ids)) return MOQE_ERR_NULL;
    if (M > 0 && (!row_ids || !perm)) return MOQE_ERR_NULL;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1); cfg.blockDim = dim3(SORT_THREADS); cfg.dynamicSmemBytes = 0; cfg.stream = (cudaStream_t)stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, route_sort_small_kernel, logits, S, E, row_offsets, M, ids, row_ids, perm, offsets) != cudaSuccess)
        return MOQE_ERR_CUDA;
    count_launch();
    return cuda_ok(cudaGetLastError());
}

extern "C" size_t moqe_permute_workspace(int M, int E) { return sort_workspace_bytes(M < 0 ? 0 : M, E); }

extern "C" moqe_status moqe_permute(const void* X_bf16, const int32_t* row_ids, int M, int C, int E, void* Xp_bf16,
                                    int32_t* perm, int32_t* offsets, void* workspace, size_t workspace_bytes,
                                    void* stream) {
    if (!offsets) return MOQE_ERR_NULL;
    if (M < 0 || E <= 0) return MOQE_ERR_SHAPE;
    if (M > 0 && (!row_ids || !perm)) return MOQE_ERR_NULL;           // an empty batch needs no row arrays
    if (M == 0) X_bf16 = Xp_bf16 = nullptr;
    if ((X_bf16 == nullptr) != (Xp_bf16 == nullptr)) return MOQE_ERR_NULL;
    if (X_bf16 && C <= 0) return MOQE_ERR_SHAPE;
    if (E > MOQE_MAX_EXPERTS) return MOQE_ERR_UNSUPPORTED;
    if (X_bf16 && (C % 8 != 0 || (uintptr_t)X_bf16 % 16 || (uintptr_t)Xp_bf16 % 16)) return MOQE_ERR_UNSUPPORTED;
    if (M > SORT_THREADS && (!workspace || workspace_bytes < sort_workspace_bytes(M, E))) return MOQE_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    moqe_status s = launch_sort(row_ids, M, E, perm, offsets, workspace, workspace_bytes, nullptr, 0, nullptr, 0, st);
    if (s != MOQE_OK || !X_bf16) return s;
    return launch_gather(X_bf16, perm, offsets + E, M, C, Xp_bf16, st);
}

extern "C" moqe_status moqe_unpermute(const void* Yp_bf16, const int32_t* perm, int M, int C, void* Y_bf16,
                                      void* stream) {
    if (!Yp_bf16 || !perm || !Y_bf16) return MOQE_ERR_NULL;
    if (M < 0 || C <= 0) return MOQE_ERR_SHAPE;
    if (C % 8 != 0 || (uintptr_t)Yp_bf16 % 16 || (uintptr_t)Y_bf16 % 16) return MOQE_ERR_UNSUPPORTED;
    if (M == 0) return MOQE_OK;
    int vec = C / 8;
    long long total = (long long)M * vec;
    move_rows_kernel<false><<<(unsigned)((total + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
        (const uint4*)Yp_bf16, perm, nullptr, M, vec, (uint4*)Y_bf16);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

// ---------------------------------------------------------------------------
// moqe_permute_static: the same sort and gather as moqe_permute for callers that
// cannot allocate device memory.  The per-block bucket totals that the
// multi-block sort needs live in a fixed array inside the library image, so this
// entry point takes no workspace and calls no allocator of any kind.
// ---------------------------------------------------------------------------
namespace moqe {
namespace {

constexpr int STATIC_SORT_MAX_ROWS = MOQE_PERMUTE_STATIC_MAX_ROWS;
constexpr int STATIC_SORT_MAX_BLOCKS = (STATIC_SORT_MAX_ROWS + SORT_THREADS - 1) / SORT_THREADS;

// [block][bucket] totals, then (after the scan) base slots.  132 KiB per device for the lifetime of
// the process.  Every entry a call reads is written by that same call first, so nothing has to be
// cleared between calls; two calls running at once on one device would overwrite each other here.
static __device__ __align__(256) int32_t g_static_sort_scratch[STATIC_SORT_MAX_BLOCKS * MAXB];

std::mutex g_static_mutex;
int32_t* g_static_scratch_addr[64] = {nullptr};

// Device address of the array on the current device.  The array's name is only a handle in host
// code; the address a kernel can use has to be asked for, once per device, with that device current.
moqe_status static_scratch(int32_t** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MOQE_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_sort_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return MOQE_ERR_CUDA;
        }
        g_static_scratch_addr[dev] = static_cast<int32_t*>(p);
    }
    *out = g_static_scratch_addr[dev];
    return MOQE_OK;
}

}  // namespace
}  // namespace moqe

extern "C" moqe_status moqe_permute_static(const void* X_bf16, const int32_t* row_ids, int M, int C, int E,
                                           void* Xp_bf16, int32_t* perm, int32_t* offsets, void* stream) {
    if (!offsets) return MOQE_ERR_NULL;
    if (M < 0 || E <= 0) return MOQE_ERR_SHAPE;
    if (M > 0 && (!row_ids || !perm)) return MOQE_ERR_NULL;
    if (M == 0) X_bf16 = Xp_bf16 = nullptr;
    if ((X_bf16 == nullptr) != (Xp_bf16 == nullptr)) return MOQE_ERR_NULL;
    if (X_bf16 && C <= 0) return MOQE_ERR_SHAPE;
    if (E > MOQE_MAX_EXPERTS) return MOQE_ERR_UNSUPPORTED;
    if (M > STATIC_SORT_MAX_ROWS) return MOQE_ERR_WORKSPACE;      // beyond the built-in scratch: use moqe_permute
    if (X_bf16 && (C % 8 != 0 || (uintptr_t)X_bf16 % 16 || (uintptr_t)Xp_bf16 % 16)) return MOQE_ERR_UNSUPPORTED;
    int32_t* scratch = nullptr;
    moqe_status s = static_scratch(&scratch);
    if (s != MOQE_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    if (M <= SORT_THREADS) {
        sort_small_kernel<<<1, SORT_THREADS, 0, st>>>(row_ids, M, E, perm, offsets, nullptr, 0, nullptr, 0, nullptr);
        count_launch();
    } else {
        int nblk = (M + SORT_THREADS - 1) / SORT_THREADS;
        sort_hist_kernel<<<nblk, SORT_THREADS, 0, st>>>(row_ids, M, E, scratch, nullptr);
        sort_scan_kernel<<<1, 1024, 0, st>>>(scratch, nblk, E, offsets);
        sort_scatter_kernel<<<nblk, SORT_THREADS, 0, st>>>(row_ids, M, E, scratch, perm, nullptr, 0);
        count_launch(3);
    }
    if (cudaGetLastError() != cudaSuccess) return MOQE_ERR_CUDA;
    if (!X_bf16) return MOQE_OK;
    return launch_gather(X_bf16, perm, offsets + E, M, C, Xp_bf16, st);
}
