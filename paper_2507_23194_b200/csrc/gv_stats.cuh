// Aggregates over the verifier's records and over latency samples: device code.
//
// The paper's metrics (Section 3.3) applied to what the Evaluator produces: a candidate is correct
// when it satisfies all unit tests (Execution Accuracy); accuracy under parallel sampling is
// reported as pass@k (Section 4.2); Speedup is the expectation over the unit tests of the ratio of
// the median reference latency to the generated kernel's latency. These are small, latency-bound
// reductions; they are written so that every floating-point operation happens in the same order
// as in the plain definition, hence results are bit-identical to the CPU oracle's.
#pragma once
#include <stdint.h>

#include "gv.h"

namespace gv {

constexpr int kStatsThreads = 256;

// results: tensor-major T x N records. pass[j] = all T tensors of candidate j have n_mismatch == 0.
// pass_at_k[k-1] = 1 - prod_{i<k} (N-c-i)/(N-i), the product taken left to right in binary64.
__global__ void __launch_bounds__(kStatsThreads) exec_summary_kernel(const gv_result* results, long long T, int N, int kmax,
                                                                     unsigned char* pass, int* n_pass, double* pass_at_k) {
    __shared__ int s_cnt;
    const int tid = threadIdx.x;
    if (tid == 0) s_cnt = 0;
    __syncthreads();
    int mine = 0;
    for (int j = tid; j < N; j += kStatsThreads) {
        bool ok = true;
        for (long long t = 0; t < T; ++t) ok = ok && results[t * N + j].n_mismatch == 0;
        pass[j] = ok ? 1 : 0;
        mine += ok ? 1 : 0;
    }
    mine = __reduce_add_sync(0xFFFFFFFFu, mine);
    if ((tid & 31) == 0 && mine) atomicAdd(&s_cnt, mine);
    __syncthreads();
    const int c = s_cnt;
    if (tid == 0) {
        *n_pass = c;
        double prod = 1.0;                       // running product: the same sequence of roundings for every k
        for (int k = 1; k <= kmax; ++k) {
            if (N - c < k) { pass_at_k[k - 1] = 1.0; continue; }
            prod = prod * (static_cast<double>(N - c - (k - 1)) / static_cast<double>(N - (k - 1)));
            pass_at_k[k - 1] = 1.0 - prod;
        }
    }
}

constexpr int kSamplesMax = 4096;

// value of rank q (0-based) among row[0..S): the x with (#smaller) <= q < (#smaller or equal)
__device__ __forceinline__ void select_ranks(const float* row, int S, int q0, int q1, float* picked /*shared, 2*/) {
    for (int a = threadIdx.x; a < S; a += kStatsThreads) {
        const float x = row[a];
        int less = 0, leq = 0;
        for (int b = 0; b < S; ++b) { less += row[b] < x; leq += row[b] <= x; }
        // Every thread that qualifies holds an equal value; equal values are bit-identical except -0 / +0,
        // so a zero is written as +0 and all writers agree on the bits.
        const float v = x == 0.0f ? 0.0f : x;
        if (less <= q0 && q0 < leq) picked[0] = v;
        if (less <= q1 && q1 < leq) picked[1] = v;
    }
}

// one CTA per unit test: medians of both sample rows and their ratio
__global__ void __launch_bounds__(kStatsThreads) median_ratio_kernel(const float* ref_lat, const float* gen_lat, int S_ref,
                                                                     int S_gen, float* median_ref, float* median_gen,
                                                                     float* ratio) {
    __shared__ float s_row[kSamplesMax];
    __shared__ float s_pick[2];
    __shared__ float s_med[2];
    const long long t = blockIdx.x;
    for (int which = 0; which < 2; ++which) {
        const int S = which == 0 ? S_ref : S_gen;
        const float* src = which == 0 ? ref_lat + t * S_ref : gen_lat + t * S_gen;
        __syncthreads();
        for (int a = threadIdx.x; a < S; a += kStatsThreads) s_row[a] = src[a];
        __syncthreads();
        select_ranks(s_row, S, (S - 1) / 2, S / 2, s_pick);
        __syncthreads();
        if (threadIdx.x == 0) s_med[which] = (S & 1) ? s_pick[0] : __fmul_rn(__fadd_rn(s_pick[0], s_pick[1]), 0.5f);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        median_ref[t] = s_med[0];
        median_gen[t] = s_med[1];
        ratio[t] = __fdiv_rn(s_med[0], s_med[1]);
    }
}

// one CTA per unit test: median latency, achieved bandwidth on the bytes the test has to move, and its
// fraction of the peak (Section 4.1 names "memory efficiency" without a formula; the header states the reading)
__global__ void __launch_bounds__(kStatsThreads) mem_efficiency_kernel(const float* lat, const unsigned long long* bytes, int S,
                                                                       double peak, float* median, double* bandwidth,
                                                                       double* efficiency) {
    __shared__ float s_row[kSamplesMax];
    __shared__ float s_pick[2];
    const long long t = blockIdx.x;
    const float* src = lat + t * S;
    for (int a = threadIdx.x; a < S; a += kStatsThreads) s_row[a] = src[a];
    __syncthreads();
    select_ranks(s_row, S, (S - 1) / 2, S / 2, s_pick);
    __syncthreads();
    if (threadIdx.x == 0) {
        const float med = (S & 1) ? s_pick[0] : __fmul_rn(__fadd_rn(s_pick[0], s_pick[1]), 0.5f);
        const double bw = __ddiv_rn(static_cast<double>(bytes[t]), static_cast<double>(med));
        median[t] = med;
        bandwidth[t] = bw;
        efficiency[t] = __ddiv_rn(bw, peak);
    }
}
// mean of T binary64 values accumulated in index order (one thread: the order is the definition)
__global__ void mean_f64_kernel(const double* x, long long T, double* mean) {
    double sum = 0.0;
    for (long long t = 0; t < T; ++t) sum += x[t];
    *mean = T ? sum / static_cast<double>(T) : 0.0;
}

// Call / execution accuracy over a (kernel x run) status matrix, K x R bytes (bit 0: compiled and ran,
// bit 1: satisfied all unit tests). First the per-kernel counts, one thread per kernel ...
__global__ void __launch_bounds__(kStatsThreads) accuracy_counts_kernel(const unsigned char* status, long long K, int R,
                                                                        int* n_call, int* n_exec) {
    const long long q = blockIdx.x * static_cast<long long>(kStatsThreads) + threadIdx.x;
    if (q >= K) return;
    int a = 0, b = 0;
    for (int r = 0; r < R; ++r) {
        const unsigned s = status[q * R + r];
        a += (s & 1u) ? 1 : 0;
        b += ((s & 3u) == 3u) ? 1 : 0;
    }
    n_call[q] = a;
    n_exec[q] = b;
}
// ... then one CTA per k = blockIdx.x + 1: pass@k(R, c) depends on the count c alone, so the R + 1 possible
// values are tabulated once (each the definition's left-to-right product), and two threads add the kernels'
// values in index order, which is the order the definition sums in.
constexpr int kRunsMax = 1024;
__global__ void __launch_bounds__(kStatsThreads) accuracy_at_k_kernel(const int* n_call, const int* n_exec, long long K, int R,
                                                                      double* call_acc, double* exec_acc) {
    __shared__ double s_pass[kRunsMax + 1];
    const int k = blockIdx.x + 1;
    for (int c = threadIdx.x; c <= R; c += kStatsThreads) {
        double v = 1.0;
        if (R - c >= k) {
            double prod = 1.0;
            for (int i = 0; i < k; ++i) prod = prod * __ddiv_rn(static_cast<double>(R - c - i), static_cast<double>(R - i));
            v = 1.0 - prod;
        }
        s_pass[c] = v;
    }
    __syncthreads();
    if (threadIdx.x == 0 || threadIdx.x == 32) {
        const int* cnt = threadIdx.x == 0 ? n_call : n_exec;
        double sum = 0.0;
        for (long long q = 0; q < K; ++q) sum += s_pass[cnt[q]];
        (threadIdx.x == 0 ? call_acc : exec_acc)[k - 1] = K ? sum / static_cast<double>(K) : 0.0;
    }
}

// the mean of the ratios, accumulated in binary64 in index order (one thread: the order is the definition)
__global__ void speedup_mean_kernel(const float* ratio, long long T, double* speedup) {
    double sum = 0.0;
    for (long long t = 0; t < T; ++t) sum += static_cast<double>(ratio[t]);
    *speedup = T ? sum / static_cast<double>(T) : 0.0;
}

}  // namespace gv
