// pipe_rates.cu -- issue rate of the instruction classes the verifier's hot loop is made of, measured
// on the GPU it runs on. Each kernel keeps 8 independent dependency chains per thread busy with one
// instruction class (inline PTX, so the assembler cannot rewrite it) on 8 resident CTAs per SM; the
// result is printed as cycles per warp-instruction per SM sub-partition (scheduler).
//
// Why it exists: the content hash the verifier must compute costs 17 add/shift/logic and 6 integer
// multiply instructions per 64-bit word. Whether the kernel is bound by DRAM or by the integer pipes
// follows from these rates (see the roofline section of the design notes), so they are measured, not
// assumed. Build and run (any sm_100a GPU):
//     nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o pipe_rates pipe_rates.cu && ./pipe_rates
// The SM clock is taken as 1.965 GHz (this part's maximum, which it holds under this load).
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#define ILP 8
#define KERNEL(name, body) \
__global__ void __launch_bounds__(256) name(uint32_t* out, uint32_t s, int iters) { \
    uint32_t x[ILP], y[ILP]; \
    for (int i = 0; i < ILP; ++i) { x[i] = s + threadIdx.x * 7 + i; y[i] = s * 3 + blockIdx.x + i * 5; } \
    uint32_t k1 = s | 1, k2 = s + 77; (void)k1; (void)k2; \
    for (int it = 0; it < iters; ++it) { \
        _Pragma("unroll") for (int i = 0; i < ILP; ++i) { body } \
    } \
    uint32_t a = 0; for (int i = 0; i < ILP; ++i) a += x[i] ^ y[i]; \
    if (a == 0x12345) out[0] = a; }
KERNEL(k_lop3, asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[i]) : "r"(y[i]), "r"(k1));)
KERNEL(k_shf, asm volatile("shf.r.wrap.b32 %0, %0, %1, 13;" : "+r"(x[i]) : "r"(y[i]));)
KERNEL(k_shr, asm volatile("shr.u32 %0, %0, 3; add.u32 %0, %0, %1;" : "+r"(x[i]) : "r"(k2));)
KERNEL(k_add, asm volatile("add.u32 %0, %0, %1;" : "+r"(x[i]) : "r"(y[i]));)
KERNEL(k_add64, asm volatile("add.cc.u32 %0, %0, %2; addc.u32 %1, %1, %3;" : "+r"(x[i]), "+r"(y[i]) : "r"(k1), "r"(k2));)
KERNEL(k_imad, asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(k1), "r"(y[i]));)
KERNEL(k_imadwide, asm volatile("{.reg .u64 t; mov.b64 t, {%0,%1}; mad.wide.u32 t, %0, %2, t; mov.b64 {%0,%1}, t;}" : "+r"(x[i]), "+r"(y[i]) : "r"(k1));)
KERNEL(k_imadhi, asm volatile("mad.hi.u32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(k1), "r"(y[i]));)
KERNEL(k_fadd, asm volatile("add.rn.f32 %0, %0, %1;" : "+r"(x[i]) : "r"(y[i]));)
KERNEL(k_ffma, asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(y[i]), "r"(k1));)
KERNEL(k_fmnmx, asm volatile("max.f32 %0, %0, %1;" : "+r"(x[i]) : "r"(y[i]));)
KERNEL(k_fmnmx3, asm volatile("max.f32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(y[i]), "r"(k1));)
KERNEL(k_setpsel, asm volatile("{.reg .pred p; setp.gt.u32 p, %0, %1; selp.u32 %0, %2, %0, p;}" : "+r"(x[i]) : "r"(y[i]), "r"(k2));)
KERNEL(k_mix_lop_imad, asm volatile("lop3.b32 %0, %0, %2, %3, 0x96; mad.lo.u32 %1, %1, %3, %2;" : "+r"(x[i]), "+r"(y[i]) : "r"(k1), "r"(k2));)
KERNEL(k_mix_lop_fadd, asm volatile("lop3.b32 %0, %0, %2, %3, 0x96; add.rn.f32 %1, %1, %2;" : "+r"(x[i]), "+r"(y[i]) : "r"(k1), "r"(k2));)
KERNEL(k_mix_imad_fadd, asm volatile("mad.lo.u32 %0, %0, %2, %3; add.rn.f32 %1, %1, %2;" : "+r"(x[i]), "+r"(y[i]) : "r"(k1), "r"(k2));)
KERNEL(k_mix3, asm volatile("lop3.b32 %0, %0, %2, %3, 0x96; mad.lo.u32 %1, %1, %3, %2; add.rn.f32 %0, %0, %3;" : "+r"(x[i]), "+r"(y[i]) : "r"(k1), "r"(k2));)
KERNEL(k_hfma2, asm volatile("fma.rn.f16x2 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(y[i]), "r"(k1));)
KERNEL(k_prmt, asm volatile("prmt.b32 %0, %0, %1, 0x5410;" : "+r"(x[i]) : "r"(y[i]));)
template <typename F> void run(const char* name, F f, int instr_per_body) {
    uint32_t* d; cudaMalloc(&d, 4);
    int iters = 4000, blocks = 148 * 8;
    f<<<blocks, 256>>>(d, 1, 10);
    cudaEvent_t a, b; cudaEventCreate(&a); cudaEventCreate(&b);
    cudaEventRecord(a); f<<<blocks, 256>>>(d, 1, iters); cudaEventRecord(b); cudaEventSynchronize(b);
    float ms; cudaEventElapsedTime(&ms, a, b);
    double warp_instr = double(blocks) * 8 * iters * ILP * instr_per_body;
    double cyc = ms * 1e-3 * 1.965e9 * 592;   // scheduler-cycles
    printf("%-16s %.3f ms  %.2f cycles per warp-instr per scheduler\n", name, ms, cyc / warp_instr);
    cudaFree(d);
}
int main() {
    run("lop3", k_lop3, 1); run("shf", k_shf, 1); run("shr+add", k_shr, 2); run("iadd", k_add, 1); run("iadd64", k_add64, 2);
    run("imad", k_imad, 1); run("imad.wide", k_imadwide, 1); run("imad.hi", k_imadhi, 1);
    run("fadd", k_fadd, 1); run("ffma", k_ffma, 1); run("fmnmx", k_fmnmx, 1); run("fmnmx3", k_fmnmx3, 1);
    run("setp+sel", k_setpsel, 2); run("hfma2", k_hfma2, 1); run("prmt", k_prmt, 1);
    run("lop3+imad", k_mix_lop_imad, 2); run("lop3+fadd", k_mix_lop_fadd, 2); run("imad+fadd", k_mix_imad_fadd, 2); run("lop+imad+fadd", k_mix3, 3);
    return 0;
}
