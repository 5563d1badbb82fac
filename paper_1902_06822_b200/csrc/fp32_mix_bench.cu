// Stand-alone instruction-mix micro-benchmark: how fast can a B200 run the inner loop of the candidate
// sweep (Section 3.4 grid search) in its scalar, saturating and packed-f32x2 forms?  Not part of
// libomse.so; built and run by `python -m paper_1902_06822_b200.fp32_mix`.  Prints, per variant,
// the time, evaluations per clock per SM (from per-block clock64 spans: an over-estimate when blocks
// do not overlap fully) and evaluations per second (from CUDA events: the figure to trust).
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>

#define MAGIC 12582912.0f

__device__ __forceinline__ unsigned long long pack2(float a, float b) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float fma_sat(float a, float b, float c) {
    float d;
    asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// MODE 0: ffma only (4 per pair)   1: clamp seq (6)   2: noclamp seq (4)   3: sat seq (5)
// MODE 4: noclamp packed f32x2     5: clamp packed (min/max scalar)   6: noclamp + fp64 flush every 64 el
// MODE 7: mixed 1 clamp slot + 7 noclamp
template <int MODE>
__global__ void __launch_bounds__(128) k(float* out, const float* xin, int n_el, int passes, long long* cyc) {
    __shared__ __align__(16) float xs[4096];
    for (int i = threadIdx.x; i < n_el; i += blockDim.x) xs[i] = xin[i];
    __syncthreads();
    float inv[8], na[8], acc[8];
    double dacc[8];
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        float a = 0.001f * (float)(threadIdx.x + 128 * s + 1);
        inv[s] = 1.0f / a; na[s] = -a; acc[s] = 0.f; dacc[s] = 0.0;
    }
    const float lo = MAGIC - 8.f, hi = MAGIC + 7.f;
    long long t0 = clock64();
    for (int p = 0; p < passes; ++p) {
        if (MODE == 4 || MODE == 5) {
            unsigned long long inv2[4], na2[4], acc2[4];
#pragma unroll
            for (int s = 0; s < 4; ++s) { inv2[s] = pack2(inv[2*s], inv[2*s+1]); na2[s] = pack2(na[2*s], na[2*s+1]); acc2[s] = pack2(acc[2*s], acc[2*s+1]); }
            const unsigned long long M2 = pack2(MAGIC, MAGIC), NM2 = pack2(-MAGIC, -MAGIC);
#pragma unroll 4
            for (int i = 0; i < n_el; i += 4) {
                float4 v = *reinterpret_cast<const float4*>(&xs[i]);
                float xe[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    unsigned long long x2 = pack2(xe[e], xe[e]);
#pragma unroll
                    for (int s = 0; s < 4; ++s) {
                        unsigned long long t = fma2(x2, inv2[s], M2);
                        if (MODE == 5) {
                            float a, b; unpack2(t, a, b);
                            a = fminf(fmaxf(a, lo), hi); b = fminf(fmaxf(b, lo), hi);
                            t = pack2(a, b);
                        }
                        unsigned long long q = add2(t, NM2);
                        unsigned long long er = fma2(na2[s], q, x2);
                        acc2[s] = fma2(er, er, acc2[s]);
                    }
                }
            }
#pragma unroll
            for (int s = 0; s < 4; ++s) unpack2(acc2[s], acc[2*s], acc[2*s+1]);
        } else {
#pragma unroll 4
            for (int i = 0; i < n_el; i += 4) {
                float4 v = *reinterpret_cast<const float4*>(&xs[i]);
                float xe[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float x = xe[e];
#pragma unroll
                    for (int s = 0; s < 8; ++s) {
                        if (MODE == 0) {
                            float t = fmaf(x, inv[s], acc[s]);
                            t = fmaf(t, inv[s], x);
                            t = fmaf(t, na[s], x);
                            acc[s] = fmaf(t, t, acc[s]);
                        } else if (MODE == 1 || (MODE == 7 && s == 0)) {
                            float t = fmaf(x, inv[s], MAGIC);
                            t = fmaxf(t, lo); t = fminf(t, hi);
                            float q = t - MAGIC;
                            float er = fmaf(na[s], q, x);
                            acc[s] = fmaf(er, er, acc[s]);
                        } else if (MODE == 2 || MODE == 6 || MODE == 7) {
                            float t = fmaf(x, inv[s], MAGIC);
                            float q = t - MAGIC;
                            float er = fmaf(na[s], q, x);
                            acc[s] = fmaf(er, er, acc[s]);
                        } else if (MODE == 3) {
                            float u = fma_sat(x, inv[s], 0.5f);
                            float t = fmaf(u, 15.f, MAGIC);
                            float q = t - (MAGIC + 8.f);
                            float er = fmaf(na[s], q, x);
                            acc[s] = fmaf(er, er, acc[s]);
                        }
                    }
                }
                if (MODE == 6 && ((i & 63) == 60)) {
#pragma unroll
                    for (int s = 0; s < 8; ++s) { dacc[s] += (double)acc[s]; acc[s] = 0.f; }
                }
            }
        }
    }
    long long t1 = clock64();
    float r = 0.f;
#pragma unroll
    for (int s = 0; s < 8; ++s) r += acc[s] + (float)dacc[s];
    out[blockIdx.x * blockDim.x + threadIdx.x] = r;
    if (threadIdx.x == 0) cyc[blockIdx.x] = t1 - t0;
}

template <int MODE>
void run(const char* name, int blocks_per_sm, float instr_per_pair) {
    int n_el = 4096, passes = 64, sms = 148;
    int blocks = sms * blocks_per_sm;
    float *out, *xin; long long* cyc;
    cudaMalloc(&out, blocks * 128 * 4); cudaMalloc(&xin, n_el * 4); cudaMalloc(&cyc, blocks * 8);
    float* h = (float*)malloc(n_el * 4);
    for (int i = 0; i < n_el; ++i) h[i] = 0.02f * (float)((i * 7919) % 1000 - 500) / 500.f;
    cudaMemcpy(xin, h, n_el * 4, cudaMemcpyHostToDevice);
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    for (int w = 0; w < 2; ++w) k<MODE><<<blocks, 128>>>(out, xin, n_el, passes, cyc);
    cudaEventRecord(e0);
    k<MODE><<<blocks, 128>>>(out, xin, n_el, passes, cyc);
    cudaEventRecord(e1); cudaEventSynchronize(e1);
    float ms; cudaEventElapsedTime(&ms, e0, e1);
    long long* hc = (long long*)malloc(blocks * 8);
    cudaMemcpy(hc, cyc, blocks * 8, cudaMemcpyDeviceToHost);
    double avg = 0; for (int i = 0; i < blocks; ++i) avg += hc[i]; avg /= blocks;
    double pairs_per_block = 128.0 * 8 * n_el * passes;
    double pairs_clk_sm = pairs_per_block * blocks_per_sm / avg;
    double pairs_s = pairs_per_block * blocks / (ms * 1e-3);
    printf("%-28s bps=%d  %.3f ms  cyc/blk=%.0f  pairs/clk/SM=%.2f  lane-instr/clk/SM=%.1f  pairs/s=%.3e  (clk~%.0f MHz) err=%s\n",
           name, blocks_per_sm, ms, avg, pairs_clk_sm, pairs_clk_sm * instr_per_pair, pairs_s, avg / (ms * 1e3),
           cudaGetErrorString(cudaGetLastError()));
    cudaFree(out); cudaFree(xin); cudaFree(cyc); free(h); free(hc);
}

int main() {
    for (int bps = 1; bps <= 4; bps *= 2) {
        run<0>("ffma x4", bps, 4);
        run<1>("clamp seq (6)", bps, 6);
        run<2>("noclamp seq (4)", bps, 4);
        run<3>("sat seq (5)", bps, 5);
        run<4>("noclamp packed f32x2", bps, 4);
        run<5>("clamp packed f32x2", bps, 6);
        run<6>("noclamp + f64 flush/64", bps, 4);
        run<7>("1 clamp + 7 noclamp", bps, 4.25);
    }
    return 0;
}
