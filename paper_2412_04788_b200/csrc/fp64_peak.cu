// Stand-alone micro-benchmark: fp64 latency (dependent chains, one warp) and throughput (many
// warps, independent chains) of the operations the performance model uses, without fused
// multiply-add.  Gives the denominator of the "alu" roofline.  Not part of libguide.so.
// Build and run: python -m paper_2412_04788_b200.fp64_peak
#include <cstdio>
#include <cuda_runtime.h>
// dependent chains: latency; many warps x independent chains: throughput
template<int OP> __global__ void chain(double* out, double a, double b, int n, long long* cyc) {
    double x0 = a + threadIdx.x, x1 = a*2+threadIdx.x, x2=a*3, x3=a*4;
    long long t0 = clock64();
    #pragma unroll 1
    for (int i = 0; i < n; i++) {
        #pragma unroll
        for (int k = 0; k < 16; k++) {
            if (OP == 0) { x0 = x0 + b; }
            if (OP == 1) { x0 = x0 * b; }
            if (OP == 2) { x0 = fma(x0, b, a); }
            if (OP == 3) { x0 = fmax(x0 * b, a); }
            if (OP == 4) { x0 = x0 + b; x1 = x1 + b; x2 = x2 + b; x3 = x3 + b; }
            if (OP == 5) { x0 = __ull2double_rn((unsigned long long)__double_as_longlong(x0) >> 3) ; }
            if (OP == 6) { x0 = x0 * b; x1 = x1 * b; x2 = x2 * b; x3 = x3 * b; }
            if (OP == 7) { x0 = a / x0; }
        }
    }
    long long t1 = clock64();
    out[blockIdx.x * blockDim.x + threadIdx.x] = x0 + x1 + x2 + x3;
    if (threadIdx.x == 0 && blockIdx.x == 0) *cyc = t1 - t0;
}
template<int OP> void run(const char* name, int blocks, int threads, int opsPerIter) {
    double* out; long long* cyc; cudaMalloc(&out, sizeof(double) * blocks * threads); cudaMalloc(&cyc, 8);
    int n = 4096;
    chain<OP><<<blocks, threads>>>(out, 1.0000001, 1.0000002, n, cyc); cudaDeviceSynchronize();
    cudaEvent_t a, b; cudaEventCreate(&a); cudaEventCreate(&b);
    cudaEventRecord(a); chain<OP><<<blocks, threads>>>(out, 1.0000001, 1.0000002, n, cyc); cudaEventRecord(b); cudaEventSynchronize(b);
    float ms; cudaEventElapsedTime(&ms, a, b); long long c; cudaMemcpy(&c, cyc, 8, cudaMemcpyDeviceToHost);
    double ops = (double)blocks * threads * n * 16 * opsPerIter;
    printf("%-28s blocks=%5d thr=%4d  cycles/op(chain, block0)=%7.2f   %.3f Top/s (thread-ops)  ms=%.3f\n", name, blocks, threads,
           (double)c / (n * 16.0), ops / ms / 1e9, ms);
    cudaFree(out); cudaFree(cyc);
}
int main() {
    run<0>("DADD dep 1 warp", 1, 32, 1);
    run<1>("DMUL dep 1 warp", 1, 32, 1);
    run<2>("DFMA dep 1 warp", 1, 32, 1);
    run<3>("DMUL+fmax dep 1 warp", 1, 32, 1);
    run<5>("shift+U64->F64 dep 1 warp", 1, 32, 1);
    run<7>("DDIV dep 1 warp", 1, 32, 1);
    run<0>("DADD dep, full", 148 * 8, 256, 1);
    run<4>("DADD 4 indep, full", 148 * 8, 256, 4);
    run<6>("DMUL 4 indep, full", 148 * 8, 256, 4);
    run<2>("DFMA dep, full", 148 * 8, 256, 1);
    run<4>("DADD 4 indep, 16 warps/SM", 148 * 2, 256, 4);
    run<4>("DADD 4 indep, 4 warps/SM", 148, 128, 4);
    run<5>("shift+U64->F64, full", 148 * 8, 256, 1);
    run<7>("DDIV, full", 148 * 8, 256, 1);
    return 0;
}
