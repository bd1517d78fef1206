// C-ABI entry points that tie the kernels together: the routed dequant-GEMM
// call, the device status word, status strings and the launch counter.
#include <atomic>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "ptx.cuh"

namespace moqe {

namespace {
std::atomic<unsigned long long> g_launches{0};
std::mutex g_status_mutex;
int* g_status_words[64] = {nullptr};
}  // namespace

void count_launch(unsigned n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int* device_status_word() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_status_mutex);
    if (!g_status_words[dev]) {
        int* p = nullptr;
        if (cudaMalloc(&p, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        if (cudaMemset(p, 0, sizeof(int)) != cudaSuccess) { cudaFree(p); return nullptr; }
        g_status_words[dev] = p;
    }
    return g_status_words[dev];
}

namespace {

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

struct WsLayout {
    size_t perm, offsets, sort, body, total;
};

WsLayout ws_layout(int M, int Np, int K, int E) {
    WsLayout w;
    size_t off = 0;
    w.perm = off;    off += align256((size_t)M * sizeof(int32_t) + 16);
    w.offsets = off; off += align256((MOQE_MAX_EXPERTS + 2) * sizeof(int32_t));
    w.sort = off;    off += align256(sort_workspace_bytes(M, E));
    w.body = off;
    size_t a = stream_workspace_bytes(M, Np, E), b = tc_workspace_bytes(M, K, E, Np), c = decode_workspace_bytes(M);
    const size_t d = dense_workspace_bytes(M, K, E, Np, (K + 127) / 128 * 128);
    a = a > b ? a : b;
    a = a > d ? a : d;
    off += align256(a > c ? a : c);
    w.total = off;
    return w;
}

constexpr int AUTO_STREAM_MAX_ROWS = 128;
constexpr int LAST_PATH = 6;

bool g_auto_decode = true;   // whether the automatic choice takes a decode kernel where it applies
bool g_auto_dense = true;    // ... and the dense-weights GEMM for large batches on small layers

// 0 = tcgen05 grouped GEMM, 1 = mma.sync streaming kernel, 2 = decode kernel, 3 = dense-weights GEMM (small layers)
int pick_kernel(int path, int M, const moqe_expert* const* ex, int E) {
    if (path == 5) return 2;
    if (path == 6) return 3;
    if (path == 1) return 1;
    if (path == 0) {
        if (g_auto_decode && decode_supported_multi(M, ex, 1, E)) return 2;
        if (M <= AUTO_STREAM_MAX_ROWS) return 1;
        return (g_auto_dense && dense_supported(M, ex[0]->N, ex[0]->K, ex, E)) ? 3 : 0;
    }
    return 0;
}

// the arrival counters at the head of the workspace body (both split-K kernels keep theirs there)
size_t body_zero_bytes(int M, int Np) {
    const size_t a = stream_zero_bytes(M, Np), b = decode_zero_bytes(M);
    return a > b ? a : b;
}

}  // namespace
}  // namespace moqe

using namespace moqe;

extern "C" size_t moqe_routed_qgemm_workspace(int M, int N, int K, int E) {
    if (M < 0 || N <= 0 || K <= 0 || E <= 0) return 0;
    int Np = (N + 127) / 128 * 128;
    return ws_layout(M, Np, K, E).total;
}

namespace {
// Argument checks shared by the single-layer entry points (`ids_or_perm`: row ids, or the sort's perm).  *done: the
// call is complete (an empty batch) when MOQE_OK comes back with it set.
moqe_status single_layer_args(const void* X, const void* ids_or_perm, const void* offsets_or_self, int M,
                              const moqe_expert* const* ex, int E, const void* Y, void* workspace, size_t workspace_bytes,
                              int path, WsLayout& w, int& kernel, bool& done) {
    done = false;
    if (!ex) return MOQE_ERR_NULL;
    if (E <= 0 || M < 0) return MOQE_ERR_SHAPE;
    if (E > MOQE_MAX_EXPERTS) return MOQE_ERR_UNSUPPORTED;
    for (int e = 0; e < E; ++e)
        if (!ex[e]) return MOQE_ERR_NULL;
    const int N = ex[0]->N, K = ex[0]->K;
    for (int e = 1; e < E; ++e)
        if (ex[e]->N != N || ex[e]->K != K) return MOQE_ERR_MISMATCH;
    if (M == 0) { done = true; return MOQE_OK; }
    if (!X || !ids_or_perm || !offsets_or_self || !Y) return MOQE_ERR_NULL;
    if (N % 8 != 0 || K % 8 != 0 || (uintptr_t)X % 16 || (uintptr_t)Y % 16) return MOQE_ERR_UNSUPPORTED;
    if (path < 0 || path > LAST_PATH) return MOQE_ERR_SHAPE;
    w = ws_layout(M, ex[0]->Np, K, E);
    if (!workspace || workspace_bytes < w.total || (uintptr_t)workspace % 256) return MOQE_ERR_WORKSPACE;
    kernel = pick_kernel(path, M, ex, E);
    if (kernel == 2 && !decode_supported_multi(M, ex, 1, E)) return MOQE_ERR_UNSUPPORTED;
    return MOQE_OK;
}

// the grouped product on sorted rows with the kernel `pick_kernel` chose
moqe_status run_sorted(int kernel, int path, const void* X, int M, const moqe_expert* const* ex, int E, void* Y,
                       const int32_t* perm, const int32_t* offsets, void* body, size_t body_bytes, cudaStream_t st) {
    const int N = ex[0]->N, K = ex[0]->K;
    if (kernel == 2) return launch_qgemm_decode_multi(&X, M, 1, ex, E, &Y, perm, offsets, body, body_bytes, st);
    if (kernel == 1) return launch_qgemm_stream(X, M, N, K, ex, E, Y, perm, offsets, body, body_bytes, st);
    if (kernel == 3) return launch_qgemm_dense(X, M, N, K, ex, E, Y, perm, offsets, body, body_bytes, st);
    tc_set_tile_tokens(path == 3 ? 128 : (path == 4 ? 256 : 0));
    return launch_qgemm_tc(X, M, N, K, ex, E, Y, perm, offsets, body, body_bytes, st);
}
}  // namespace

extern "C" moqe_status moqe_routed_qgemm_path(const void* X_bf16, const int32_t* row_ids, int M,
                                              const moqe_expert* const* h_experts, int E, void* Y_bf16, void* workspace,
                                              size_t workspace_bytes, void* stream, int path) {
    WsLayout w;
    int kernel = 0;
    bool done = false;
    moqe_status s = single_layer_args(X_bf16, row_ids, row_ids, M, h_experts, E, Y_bf16, workspace, workspace_bytes, path, w, kernel, done);
    if (s != MOQE_OK || done) return s;
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)workspace;
    int32_t* perm = (int32_t*)(base + w.perm);
    int32_t* offsets = (int32_t*)(base + w.offsets);
    const size_t zero_bytes = kernel != 0 ? body_zero_bytes(M, h_experts[0]->Np) : 0;
    s = launch_sort(row_ids, M, E, perm, offsets, base + w.sort, w.body - w.sort, base + w.body, zero_bytes, Y_bf16,
                    h_experts[0]->N, st);
    if (s != MOQE_OK) return s;
    return run_sorted(kernel, path, X_bf16, M, h_experts, E, Y_bf16, perm, offsets, base + w.body, w.total - w.body, st);
}

extern "C" moqe_status moqe_routed_qgemm_sorted(const void* X_bf16, const int32_t* perm, const int32_t* offsets, int M,
                                                const moqe_expert* const* h_experts, int E, void* Y_bf16, void* workspace,
                                                size_t workspace_bytes, void* stream, int path) {
    WsLayout w;
    int kernel = 0;
    bool done = false;
    moqe_status s = single_layer_args(X_bf16, perm, offsets, M, h_experts, E, Y_bf16, workspace, workspace_bytes, path, w, kernel, done);
    if (s != MOQE_OK || done) return s;
    char* base = (char*)workspace;
    return run_sorted(kernel, path, X_bf16, M, h_experts, E, Y_bf16, perm, offsets, base + w.body, w.total - w.body,
                      (cudaStream_t)stream);
}

extern "C" moqe_status moqe_routed_qgemm_sorted_multi(const void* const* h_X_bf16, const int32_t* perm, const int32_t* offsets,
                                                      int M, int n_layers, const moqe_expert* const* h_experts, int E,
                                                      void* const* h_Y_bf16, void* workspace, size_t workspace_bytes,
                                                      void* stream) {
    if (!h_experts || !h_X_bf16 || !h_Y_bf16) return MOQE_ERR_NULL;
    if (E <= 0 || M < 0 || n_layers <= 0) return MOQE_ERR_SHAPE;
    if (n_layers * E > MOQE_MAX_EXPERTS) return MOQE_ERR_UNSUPPORTED;
    for (int l = 0; l < n_layers; ++l) {
        for (int e = 0; e < E; ++e)
            if (!h_experts[l * E + e]) return MOQE_ERR_NULL;
        const int N = h_experts[l * E]->N, K = h_experts[l * E]->K;
        for (int e = 1; e < E; ++e)
            if (h_experts[l * E + e]->N != N || h_experts[l * E + e]->K != K) return MOQE_ERR_MISMATCH;
        if (M > 0 && (!h_X_bf16[l] || !h_Y_bf16[l])) return MOQE_ERR_NULL;
        if (N % 8 != 0 || K % 8 != 0 || (uintptr_t)h_X_bf16[l] % 16 || (uintptr_t)h_Y_bf16[l] % 16) return MOQE_ERR_UNSUPPORTED;
    }
    if (M == 0) return MOQE_OK;
    if (!perm || !offsets) return MOQE_ERR_NULL;
    if (!decode_supported_multi(M, h_experts, n_layers, E)) return MOQE_ERR_UNSUPPORTED;
    WsLayout w = ws_layout(M, h_experts[0]->Np, h_experts[0]->K, E);
    if (!workspace || workspace_bytes < w.total || (uintptr_t)workspace % 256) return MOQE_ERR_WORKSPACE;
    char* base = (char*)workspace;
    return launch_qgemm_decode_multi(h_X_bf16, M, n_layers, h_experts, E, h_Y_bf16, perm, offsets, base + w.body,
                             w.total - w.body, (cudaStream_t)stream);
}

namespace {
// shared argument checks of the decode-only fused entry points
moqe_status fused_args(const void* X, const int32_t* perm, const int32_t* offsets, int M, const moqe_expert* const* ex, int E,
                       const void* Y, void* workspace, size_t workspace_bytes, size_t& body, size_t& total) {
    if (!ex) return MOQE_ERR_NULL;
    if (E <= 0 || M < 0) return MOQE_ERR_SHAPE;
    if (E > MOQE_MAX_EXPERTS) return MOQE_ERR_UNSUPPORTED;
    for (int e = 0; e < E; ++e)
        if (!ex[e]) return MOQE_ERR_NULL;
    const int N = ex[0]->N, K = ex[0]->K;
    for (int e = 1; e < E; ++e)
        if (ex[e]->N != N || ex[e]->K != K) return MOQE_ERR_MISMATCH;
    if (M == 0) return MOQE_OK;
    if (!X || !perm || !offsets || !Y) return MOQE_ERR_NULL;
    if (N % 8 != 0 || K % 8 != 0 || (uintptr_t)X % 16 || (uintptr_t)Y % 16) return MOQE_ERR_UNSUPPORTED;
    if (!decode_supported_multi(M, ex, 1, E)) return MOQE_ERR_UNSUPPORTED;
    WsLayout w = ws_layout(M, ex[0]->Np, K, E);
    if (!workspace || workspace_bytes < w.total || (uintptr_t)workspace % 256) return MOQE_ERR_WORKSPACE;
    body = w.body;
    total = w.total;
    return MOQE_OK;
}
}  // namespace

extern "C" moqe_status moqe_routed_qgemm_sorted_gated(const void* X_bf16, const int32_t* perm, const int32_t* offsets, int M,
                                                      const moqe_expert* const* h_gate, const moqe_expert* const* h_up, int E,
                                                      void* Y_bf16, void* workspace, size_t workspace_bytes, void* stream) {
    if (!h_up) return MOQE_ERR_NULL;
    size_t body = 0, total = 0;
    moqe_status s = fused_args(X_bf16, perm, offsets, M, h_gate, E, Y_bf16, workspace, workspace_bytes, body, total);
    if (s != MOQE_OK || M == 0) return s;
    for (int e = 0; e < E; ++e)
        if (!h_up[e]) return MOQE_ERR_NULL;
    return launch_qgemm_decode_ext(&X_bf16, M, 1, h_gate, h_up, E, &Y_bf16, nullptr, perm, offsets, (char*)workspace + body,
                                   total - body, (cudaStream_t)stream);
}

extern "C" moqe_status moqe_routed_qgemm_sorted_residual(const void* X_bf16, const int32_t* perm, const int32_t* offsets, int M,
                                                         const moqe_expert* const* h_experts, int E, const void* R_bf16,
                                                         void* Y_bf16, void* workspace, size_t workspace_bytes, void* stream) {
    size_t body = 0, total = 0;
    moqe_status s = fused_args(X_bf16, perm, offsets, M, h_experts, E, Y_bf16, workspace, workspace_bytes, body, total);
    if (s != MOQE_OK || M == 0) return s;
    if (!R_bf16) return MOQE_ERR_NULL;
    return launch_qgemm_decode_ext(&X_bf16, M, 1, h_experts, nullptr, E, &Y_bf16, &R_bf16, perm, offsets,
                                   (char*)workspace + body, total - body, (cudaStream_t)stream);
}

extern "C" moqe_status moqe_routed_qgemm_workspace_clear(void* workspace, size_t workspace_bytes, int M, int N, int K,
                                                         int E, void* stream) {
    if (M < 0 || N <= 0 || K <= 0 || E <= 0) return MOQE_ERR_SHAPE;
    const int Np = (N + 127) / 128 * 128;
    WsLayout w = ws_layout(M, Np, K, E);
    if (!workspace || workspace_bytes < w.total || (uintptr_t)workspace % 256) return MOQE_ERR_WORKSPACE;
    size_t zb = body_zero_bytes(M, Np);
    if (zb == 0) return MOQE_OK;
    return cuda_ok(cudaMemsetAsync((char*)workspace + w.body, 0, zb, (cudaStream_t)stream));
}

extern "C" moqe_status moqe_routed_qgemm(const void* X_bf16, const int32_t* row_ids, int M,
                                         const moqe_expert* const* h_experts, int E, void* Y_bf16, void* workspace,
                                         size_t workspace_bytes, void* stream) {
    return moqe_routed_qgemm_path(X_bf16, row_ids, M, h_experts, E, Y_bf16, workspace, workspace_bytes, stream, 0);
}

extern "C" moqe_status moqe_tune(const char* key, int value) {
    if (!key) return MOQE_ERR_NULL;
    if (!strcmp(key, "stream_tile_cost_w8")) { stream_set_tile_cost(8, value); return MOQE_OK; }
    if (!strcmp(key, "stream_tile_cost_w4")) { stream_set_tile_cost(4, value); return MOQE_OK; }
    if (!strcmp(key, "stream_tile_cost_w3")) { stream_set_tile_cost(3, value); return MOQE_OK; }
    if (!strcmp(key, "auto_decode")) { g_auto_decode = value != 0; return MOQE_OK; }
    if (!strcmp(key, "auto_dense")) { g_auto_dense = value != 0; return MOQE_OK; }
    if (!strcmp(key, "decode_tile_cost_w8")) { decode_set_tile_cost(8, value); return MOQE_OK; }
    if (!strcmp(key, "decode_tile_cost_w4")) { decode_set_tile_cost(4, value); return MOQE_OK; }
    if (!strcmp(key, "decode_tile_cost_w3")) { decode_set_tile_cost(3, value); return MOQE_OK; }
    return MOQE_ERR_UNSUPPORTED;
}

extern "C" moqe_status moqe_async_status(void* stream) {
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return MOQE_ERR_CUDA;
    int* w = device_status_word();
    if (!w) return MOQE_ERR_ALLOC;
    int v = 0;
    if (cudaMemcpy(&v, w, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return MOQE_ERR_CUDA;
    if (v != 0 && cudaMemset(w, 0, sizeof(int)) != cudaSuccess) return MOQE_ERR_CUDA;
    return (moqe_status)v;
}

namespace moqe {
namespace {
// One thread initialises an mbarrier on which nobody ever arrives and waits for it with the library's bounded wait.
__global__ void selftest_timeout_kernel(int* status, unsigned long long limit_ns, int* returned) {
    __shared__ unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const bool ok = mbar_wait_limit(smem_u32(&bar), 0u, &abort_flag, status, limit_ns);
        *returned = ok ? 1 : 2;
    }
}
}  // namespace
}  // namespace moqe

extern "C" moqe_status moqe_selftest_timeout(unsigned limit_us, int* d_returned, void* stream) {
    if (!d_returned) return MOQE_ERR_NULL;
    if (limit_us == 0 || limit_us > 1000000u) return MOQE_ERR_SHAPE;
    int* w = device_status_word();
    if (!w) return MOQE_ERR_ALLOC;
    selftest_timeout_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(w, (unsigned long long)limit_us * 1000ull, d_returned);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

extern "C" const char* moqe_status_str(moqe_status s) {
    switch (s) {
        case MOQE_OK: return "ok";
        case MOQE_ERR_NULL: return "a required pointer is NULL";
        case MOQE_ERR_SHAPE: return "bad or inconsistent size";
        case MOQE_ERR_UNSUPPORTED: return "unsupported format, size or alignment";
        case MOQE_ERR_ALLOC: return "device allocation failed";
        case MOQE_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case MOQE_ERR_MISMATCH: return "experts disagree on N or K";
        case MOQE_ERR_CUDA: return "a CUDA call failed";
        case MOQE_ERR_EXPERT_ID: return "an expert id outside [0,E) was seen on the device";
        case MOQE_ERR_TIMEOUT: return "a bounded in-kernel wait ran out";
        case MOQE_ERR_IO: return "file missing, unreadable, unwritable or not a whole expert image";
    }
    return "unknown status";
}

extern "C" unsigned long long moqe_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
