// fp32 CUDA-core kernels, NCHW.  Used by graphs compiled with XENOS_PRECISION_FP32_CUDA_CORE:
// one kernel per fused operator (unlinked execution) and one kernel for the linked chain
// ConvX -> Conv1x1 -> ZPooling (Table 1 of the Xenos paper), where the intermediate feature
// maps of a tile stay in shared memory in the order the next stage reads them.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace xk {

__device__ __forceinline__ float apply_act(float v, int act) {
    if (act >= 1) v = fmaxf(v, 0.0f);
    if (act == 2) v = fminf(v, 6.0f);
    return v;
}

// Direct convolution: y[n][k][p][q] = b[k] + sum_{c,r,s} x[n][g*Cg + c][p*st - pad + r][q*st - pad + s] * w[k][c][r][s],
// one output element per thread, then the fused activation.
__global__ void f32_conv_kernel(const float *__restrict__ x, const float *__restrict__ w,
                                const float *__restrict__ b, float *__restrict__ y, int N, int C, int H,
                                int W, int K, int P, int Q, int k, int stride, int pad, int groups, int act) {
    long long total = (long long)N * K * P * Q;
    int Cg = C / groups, Kg = K / groups;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        int q = (int)(i % Q);
        long long t = i / Q;
        int p = (int)(t % P); t /= P;
        int kk = (int)(t % K);
        int n = (int)(t / K);
        int g = kk / Kg;
        float acc = 0.0f;
        for (int c = 0; c < Cg; ++c) {
            const float *xc = x + ((size_t)n * C + (size_t)g * Cg + c) * H * W;
            const float *wc = w + ((size_t)kk * Cg + c) * k * k;
            for (int r = 0; r < k; ++r) {
                int ih = p * stride - pad + r;
                if (ih < 0 || ih >= H) continue;
                for (int s = 0; s < k; ++s) {
                    int iw = q * stride - pad + s;
                    if (iw < 0 || iw >= W) continue;
                    acc = fmaf(xc[(size_t)ih * W + iw], wc[r * k + s], acc);
                }
            }
        }
        y[i] = apply_act(acc + b[kk], act);
    }
}

// Max (kind 0) or average (kind 1, divisor = in-range elements) pooling.
__global__ void f32_pool_kernel(const float *__restrict__ x, float *__restrict__ y, int N, int C, int H, int W,
                                int P, int Q, int k, int stride, int pad, int kind) {
    long long total = (long long)N * C * P * Q;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        int q = (int)(i % Q);
        long long t = i / Q;
        int p = (int)(t % P); t /= P;
        const float *xc = x + (size_t)t * H * W;
        float m = -INFINITY, acc = 0.0f;
        int cnt = 0;
        for (int r = 0; r < k; ++r) {
            int ih = p * stride - pad + r;
            if (ih < 0 || ih >= H) continue;
            for (int s = 0; s < k; ++s) {
                int iw = q * stride - pad + s;
                if (iw < 0 || iw >= W) continue;
                float v = xc[(size_t)ih * W + iw];
                m = fmaxf(m, v);
                acc += v;
                ++cnt;
            }
        }
        y[i] = kind == 0 ? m : (cnt ? acc / (float)cnt : 0.0f);
    }
}

// Global average: one warp per (image, channel), fixed-order lane sums then a shuffle tree.
__global__ void f32_gap_kernel(const float *__restrict__ x, float *__restrict__ y, int NC, int HW) {
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= NC) return;
    const float *xi = x + (size_t)warp * HW;
    float acc = 0.0f;
    for (int i = lane; i < HW; i += 32) acc += xi[i];
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) y[warp] = acc / (float)HW;
}

__global__ void f32_add_kernel(const float *__restrict__ a, const float *__restrict__ b, float *__restrict__ y,
                               long long n, int act) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        y[i] = apply_act(a[i] + b[i], act);
}

// x.mul (c == nullptr) / x.mac: the product is rounded before the sum (no fused multiply-add).
__global__ void f32_mulmac_kernel(const float *__restrict__ a, const float *__restrict__ b, const float *__restrict__ c,
                                  float *__restrict__ y, long long n) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const float p = __fmul_rn(a[i], b[i]);
        y[i] = c ? __fadd_rn(p, c[i]) : p;
    }
}

// x.split, one part: y [N][Ci][HW] = x [N][Ctot][HW] at channel offset coff.
__global__ void f32_slice_kernel(const float *__restrict__ x, float *__restrict__ y, int N, int Ci, int HW,
                                 int Ctot, int coff) {
    long long per = (long long)Ci * HW, total = (long long)N * per;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        long long n = i / per, r = i % per;
        y[i] = x[(n * Ctot + coff) * HW + r];
    }
}

// One concat input: x [N][Ci][HW] -> y [N][Ctot][HW] at channel offset coff.
__global__ void f32_concat_part_kernel(const float *__restrict__ x, float *__restrict__ y, int N, int Ci, int HW,
                                       int Ctot, int coff) {
    long long per = (long long)Ci * HW, total = (long long)N * per;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        long long n = i / per, r = i % per;
        y[(n * Ctot + coff) * HW + r] = x[i];
    }
}

// y = W x + B (Eq. 1), one output per thread.
__global__ void f32_fc_kernel(const float *__restrict__ x, const float *__restrict__ w, const float *__restrict__ b,
                              float *__restrict__ y, int N, int C, int K, int act) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * K) return;
    int n = i / K, k = i % K;
    float acc = 0.0f;
    for (int c = 0; c < C; ++c) acc = fmaf(w[(size_t)k * C + c], x[(size_t)n * C + c], acc);
    y[i] = apply_act(acc + b[k], act);
}

// ------------------------------------------------------------------------------------------------
// Linked chain ConvX(+act) -> Conv1x1(+act) -> pool, one CTA per (image, outC part, pool tile).
//   stage 0: the input patch the tile needs goes to shared memory, zero-filled outside the image
//   stage 1: ConvX on the patch -> shared memory [Cmid][rh][rw], i.e. channel-major so that
//            stage 2 reads a pixel's channels at a fixed stride and neighbouring threads read
//            neighbouring pixels (the consumer's read order)
//   stage 2: Conv1x1 over the CTA's slice of output channels, pooled in registers
// Every index is checked against the buffer extents; a failed check sets the status word and
// skips the access.
// ------------------------------------------------------------------------------------------------
struct F32ChainParams {
    const float *x, *w1, *b1, *w2, *b2;
    float *y;
    int N, C, H, W;          // input
    int Cmid, P, Q;          // stage-1 output
    int k, stride, pad, act1;
    int K2, act2;
    int pool_kind, pool_k, pool_stride, PP, PQ;
    int parts_outc, tile_h, tile_w, tiles_h, tiles_w, halo_h, halo_w;
    unsigned int *status;
};

__global__ void f32_conv_conv_pool_kernel(F32ChainParams p) {
    extern __shared__ float smem[];
    int cta = blockIdx.x;
    int tx = cta % p.tiles_w; cta /= p.tiles_w;
    int ty = cta % p.tiles_h; cta /= p.tiles_h;
    int part = cta % p.parts_outc;
    int n = cta / p.parts_outc;
    if (n >= p.N) return;
    // pool tile -> stage-1 patch -> input patch
    int py0 = ty * p.tile_h, px0 = tx * p.tile_w;
    int th = min(p.tile_h, p.PP - py0), tw = min(p.tile_w, p.PQ - px0);
    int rh = (th - 1) * p.pool_stride + p.pool_k, rw = (tw - 1) * p.pool_stride + p.pool_k;
    int r0 = py0 * p.pool_stride, c0 = px0 * p.pool_stride;                 // stage-1 origin (pool pad is 0)
    int ih = (rh - 1) * p.stride + p.k, iw = (rw - 1) * p.stride + p.k;
    int i0 = r0 * p.stride - p.pad, j0 = c0 * p.stride - p.pad;             // input origin, may be negative
    int max_ih = (p.halo_h - 1) * p.stride + p.k, max_iw = (p.halo_w - 1) * p.stride + p.k;
    float *s_in = smem;                                                      // [C][ih][iw]
    float *s_mid = smem + (size_t)p.C * max_ih * max_iw;                     // [Cmid][rh][rw]
    if (rh > p.halo_h || rw > p.halo_w || ih > max_ih || iw > max_iw) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0u, 0x80000000u | 10u);
        return;
    }
    for (int i = threadIdx.x; i < p.C * ih * iw; i += blockDim.x) {
        int c = i / (ih * iw), r = i % (ih * iw);
        int a = i0 + r / iw, b = j0 + r % iw;
        float v = 0.0f;
        if (a >= 0 && a < p.H && b >= 0 && b < p.W) v = p.x[(((size_t)n * p.C + c) * p.H + a) * p.W + b];
        s_in[i] = v;
    }
    __syncthreads();
    // stage 1: one (channel, pixel) per thread-iteration; pixels fastest so threads read s_in contiguously
    for (int i = threadIdx.x; i < p.Cmid * rh * rw; i += blockDim.x) {
        int m = i / (rh * rw), r = i % (rh * rw);
        int a = r / rw, b = r % rw;
        float acc = 0.0f;
        const float *wm = p.w1 + (size_t)m * p.C * p.k * p.k;
        for (int c = 0; c < p.C; ++c) {
            const float *sc = s_in + ((size_t)c * ih + a * p.stride) * iw + b * p.stride;
            const float *wc = wm + c * p.k * p.k;
            for (int r1 = 0; r1 < p.k; ++r1)
                for (int s1 = 0; s1 < p.k; ++s1) acc = fmaf(sc[r1 * iw + s1], wc[r1 * p.k + s1], acc);
        }
        // positions of the patch outside the stage-1 extent are never read by a pool window
        s_mid[i] = apply_act(acc + p.b1[m], p.act1);
    }
    __syncthreads();
    // stage 2 + pool: one (output channel, pool output) per thread-iteration
    int kper = p.K2 / p.parts_outc, k0 = part * kper;
    for (int i = threadIdx.x; i < kper * th * tw; i += blockDim.x) {
        int kk = k0 + i / (th * tw), r = i % (th * tw);
        int oy = r / tw, ox = r % tw;
        const float *w2 = p.w2 + (size_t)kk * p.Cmid;
        float bias = p.b2[kk];
        float m = -INFINITY, sum = 0.0f;
        for (int dy = 0; dy < p.pool_k; ++dy)
            for (int dx = 0; dx < p.pool_k; ++dx) {
                int a = oy * p.pool_stride + dy, b = ox * p.pool_stride + dx;
                float acc = 0.0f;
                for (int c = 0; c < p.Cmid; ++c) acc = fmaf(s_mid[((size_t)c * rh + a) * rw + b], w2[c], acc);
                float v = apply_act(acc + bias, p.act2);
                m = fmaxf(m, v);
                sum += v;
            }
        float o = p.pool_kind == 0 ? m : sum / (float)(p.pool_k * p.pool_k);
        size_t oi = (((size_t)n * p.K2 + kk) * p.PP + (py0 + oy)) * p.PQ + (px0 + ox);
        p.y[oi] = o;
    }
}

}  // namespace xk
