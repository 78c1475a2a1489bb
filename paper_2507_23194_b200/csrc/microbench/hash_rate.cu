// hash_rate.cu -- throughput of the content hash's mixing function alone (operands in registers, no
// memory traffic), in several formulations that move part of the shifts/additions from the
// add/shift/logic pipe to the integer-multiply pipe. Printed as cycles per warp-hash per SM
// sub-partition and as the equivalent GB/s of hashed data for the whole GPU: the ceiling the verifier
// would reach if it did nothing but hash. Build (from this directory) and run:
//     nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -I.. -I../../../include -o hash_rate hash_rate.cu && ./hash_rate
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#include "gv_device.cuh"
using namespace gv;
template <int MASK, int ILP>
__global__ void __launch_bounds__(256) k(uint64_t* out, uint32_t seed, int iters) {
    uint32_t lo[ILP], hi[ILP];
    HashConsts hc; hc.init();
    for (int i = 0; i < ILP; ++i) { lo[i] = seed + threadIdx.x * 7 + i; hi[i] = blockIdx.x + i * 3; }
    uint64_t acc = 0;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < ILP; ++i) {
            uint64_t h = splitmix64_split<MASK>(lo[i] ^ it, hi[i], hc.one, hc.p2, hc.p5, hc.p1);
            acc += h;
            lo[i] = (uint32_t)h; hi[i] = (uint32_t)(h >> 32);
        }
    }
    if (acc == 0x1234567) out[0] = acc;
}
template <int MASK, int ILP>
void run(const char* name) {
    uint64_t* d; cudaMalloc(&d, 8);
    int iters = 2000;
    int blocks = 148 * 8;
    k<MASK, ILP><<<blocks, 256>>>(d, 1, 10);
    cudaEvent_t a, b; cudaEventCreate(&a); cudaEventCreate(&b);
    cudaEventRecord(a);
    k<MASK, ILP><<<blocks, 256>>>(d, 1, iters);
    cudaEventRecord(b); cudaEventSynchronize(b);
    float ms; cudaEventElapsedTime(&ms, a, b);
    double hashes = double(blocks) * 256 * iters * ILP;
    double per_sched_cycle = (ms * 1e-3 * 1.95e9) / (hashes / 32 / 592);
    printf("%s mask=%d ilp=%d: %.3f ms, %.2f Ghash/s, %.1f cycles per warp-hash per scheduler -> %.2f TB/s hash-only\n", name, MASK, ILP, ms,
           hashes / ms / 1e6, per_sched_cycle, hashes * 8 / ms / 1e9);
    cudaFree(d);
}
int main() {
    run<0, 2>("plain"); run<0, 4>("plain");
    run<1, 4>("x30"); run<2, 4>("x27"); run<4, 4>("x31"); run<3, 4>("x30+27"); run<5, 4>("x30+31"); run<7, 4>("all3");
    run<8, 4>("add"); run<9, 4>("add+x30"); run<11, 4>("add+x30+27"); run<15, 4>("all");
    return 0;
}
