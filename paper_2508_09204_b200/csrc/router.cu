// Router front end on the device: per-sample mean of the activation rows -> two-layer MLP (ReLU, no biases) -> one score
// per expert -> arg-max, so that expert ids never leave the GPU; and the load report of a routed batch (mean routing
// probability P_i, dispatched fraction F_i, balance term L_bal = N * sum P_i * F_i).
//
// Section 3.2 of the paper ("Router Model"): the router ends in an MLP that maps a feature vector of the sample to the
// routing logits and one expert index leaves it; the paper's trained encoders are not reproduced -- the feature vector
// here is the mean of the sample's rows.  Section 3.3 ("Router Fine-Tuning") defines P_i, F_i and L_bal.
//
// Everything is fp32 with a fixed summation order (no atomics on floats): the same call gives the same bits.
#include "common.cuh"

namespace moqe {
namespace {

constexpr int POOL_THREADS = 256;     // 8 warps: warp w sums the rows r = w (mod 8) of the sample, lane l the features 8l .. 8l + 7
constexpr int POOL_H = 256;           // features per block

// pooled[s][h] = (1 / n_s) * sum of the sample's rows
__global__ void __launch_bounds__(POOL_THREADS) router_pool_kernel(const uint16_t* __restrict__ X, const int32_t* __restrict__ row_offsets,
                                                                   int H, float* __restrict__ pooled) {
    __shared__ float s_part[8][POOL_H];
    const int s = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h0 = blockIdx.x * POOL_H + lane * 8;
    const int r0 = row_offsets[s], r1 = row_offsets[s + 1];
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (h0 < H) {
#pragma unroll 4
        for (int r = r0 + warp; r < r1; r += 8) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(X + (size_t)r * H + h0));
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                acc[2 * i] += __uint_as_float(w[i] << 16);
                acc[2 * i + 1] += __uint_as_float(w[i] & 0xFFFF0000u);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) s_part[warp][lane * 8 + i] = acc[i];
    __syncthreads();
    const int h = blockIdx.x * POOL_H + threadIdx.x;
    if (h < H) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) t += s_part[w][threadIdx.x];       // warp order: deterministic
        pooled[(size_t)s * H + h] = r1 > r0 ? t / (float)(r1 - r0) : 0.f;
    }
}

// hidden[s][d] = max(0, pooled[s] . W1[d]); one warp per (d, s)
__global__ void __launch_bounds__(256) router_hidden_kernel(const float* __restrict__ pooled, const float* __restrict__ W1, int S, int H,
                                                            int D, float* __restrict__ hidden) {
    const int lane = threadIdx.x & 31;
    const long long wid = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (wid >= (long long)S * D) return;
    const int s = (int)(wid / D), d = (int)(wid % D);
    const float* p = pooled + (size_t)s * H;
    const float* w = W1 + (size_t)d * H;
    float acc = 0.f;
    for (int h = lane * 4; h < H; h += 128) {
        if (h + 4 <= H) {
            const float4 a = *reinterpret_cast<const float4*>(p + h), b = __ldg(reinterpret_cast<const float4*>(w + h));
            acc = fmaf(a.x, b.x, acc); acc = fmaf(a.y, b.y, acc); acc = fmaf(a.z, b.z, acc); acc = fmaf(a.w, b.w, acc);
        } else {
            for (int j = h; j < H; ++j) acc = fmaf(p[j], w[j], acc);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) hidden[(size_t)s * D + d] = fmaxf(acc, 0.f);
}

// logits[s][e] = hidden[s] . W2[e]; id = first maximum (NaN never wins; all-NaN -> 0); one warp per sample
__global__ void __launch_bounds__(256) router_logits_kernel(const float* __restrict__ hidden, const float* __restrict__ W2, int S, int D, int E,
                                                            float* __restrict__ logits, int32_t* __restrict__ ids) {
    const int lane = threadIdx.x & 31;
    const int s = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (s >= S) return;
    const float* hdn = hidden + (size_t)s * D;
    float best = 0.f;
    int arg = -1;
    for (int e = 0; e < E; ++e) {
        const float* w = W2 + (size_t)e * D;
        float acc = 0.f;
        for (int d = lane; d < D; d += 32) acc = fmaf(hdn[d], __ldg(w + d), acc);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) logits[(size_t)s * E + e] = acc;
        if (acc == acc && (arg < 0 || acc > best)) { best = acc; arg = e; }
    }
    if (lane == 0) ids[s] = arg < 0 ? 0 : arg;
}

// one block: thread e owns expert e
__global__ void __launch_bounds__(64) router_report_kernel(const float* __restrict__ logits, const int32_t* __restrict__ ids, int S, int E,
                                                           float* __restrict__ report, int32_t* __restrict__ counts) {
    __shared__ float s_pf[MOQE_MAX_EXPERTS];
    const int e = threadIdx.x;
    float P = 0.f, F = 0.f;
    if (e < E) {
        int n = 0;
        for (int s = 0; s < S; ++s) {
            const float* l = logits + (size_t)s * E;
            float mx = l[0];
            for (int j = 1; j < E; ++j) mx = fmaxf(mx, l[j]);
            float den = 0.f;
            for (int j = 0; j < E; ++j) den += expf(l[j] - mx);
            P += expf(l[e] - mx) / den;
            n += ids[s] == e ? 1 : 0;
        }
        P /= (float)S;
        F = (float)n / (float)S;
        report[e] = P;
        report[E + e] = F;
        if (counts) counts[e] = n;
        s_pf[e] = P * F;
    }
    __syncthreads();
    if (e == 0) {
        float t = 0.f;
        for (int j = 0; j < E; ++j) t += s_pf[j];
        report[2 * E] = (float)E * t;
    }
}

size_t align256r(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace
}  // namespace moqe

using namespace moqe;

extern "C" size_t moqe_router_mlp_workspace(int S, int H, int D) {
    if (S < 0 || H <= 0 || D <= 0) return 0;
    return align256r((size_t)S * H * sizeof(float)) + align256r((size_t)S * D * sizeof(float));
}

extern "C" moqe_status moqe_router_mlp(const void* X_bf16, const int32_t* row_offsets, int S, int H, const float* W1, int D,
                                       const float* W2, int E, float* logits, int32_t* ids, void* workspace,
                                       size_t workspace_bytes, void* stream) {
    if (S < 0 || H <= 0 || D <= 0 || E <= 0) return MOQE_ERR_SHAPE;
    if (E > MOQE_MAX_EXPERTS || H % 8 != 0) return MOQE_ERR_UNSUPPORTED;
    if (S == 0) return MOQE_OK;
    if (!X_bf16 || !row_offsets || !W1 || !W2 || !logits || !ids) return MOQE_ERR_NULL;
    if ((uintptr_t)X_bf16 % 16 || (uintptr_t)W1 % 16) return MOQE_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < moqe_router_mlp_workspace(S, H, D) || (uintptr_t)workspace % 256) return MOQE_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    float* pooled = (float*)workspace;
    float* hidden = (float*)((char*)workspace + align256r((size_t)S * H * sizeof(float)));
    router_pool_kernel<<<dim3((H + POOL_H - 1) / POOL_H, S), POOL_THREADS, 0, st>>>((const uint16_t*)X_bf16, row_offsets, H, pooled);
    const long long warps = (long long)S * D;
    router_hidden_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(pooled, W1, S, H, D, hidden);
    router_logits_kernel<<<(S + 7) / 8, 256, 0, st>>>(hidden, W2, S, D, E, logits, ids);
    count_launch(3);
    return cuda_ok(cudaGetLastError());
}

extern "C" moqe_status moqe_router_load_report(const float* logits, const int32_t* ids, int S, int E, float* report,
                                               int32_t* counts, void* stream) {
    if (S <= 0 || E <= 0) return MOQE_ERR_SHAPE;
    if (E > MOQE_MAX_EXPERTS) return MOQE_ERR_UNSUPPORTED;
    if (!logits || !ids || !report) return MOQE_ERR_NULL;
    router_report_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(logits, ids, S, E, report, counts);
    count_launch();
    return cuda_ok(cudaGetLastError());
}
