// bf16 NHWC CUDA-core kernels for the operators that are not contractions: depthwise 3x3,
// pooling, global average, residual add and concat (x.conv depthwise, x.gampool, x.add, x.concat
// of Table 3).  Each thread moves 8 channels (one 128-bit access) so a warp touches 512
// contiguous bytes of a pixel's channel vector; arithmetic is fp32, storage rounds to nearest even.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels_f32.cuh"

namespace xk {

struct f8 { float v[8]; };

__device__ __forceinline__ f8 unpack8(const uint4 &u) {
    f8 r;
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        r.v[2 * i] = __uint_as_float(w[i] << 16);
        r.v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    return r;
}

__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);   // .x = a (low half), .y = b
    return *reinterpret_cast<uint32_t *>(&h);
}

__device__ __forceinline__ uint4 pack8(const f8 &r) {
    uint4 u;
    u.x = pack2(r.v[0], r.v[1]); u.y = pack2(r.v[2], r.v[3]);
    u.z = pack2(r.v[4], r.v[5]); u.w = pack2(r.v[6], r.v[7]);
    return u;
}

// Depthwise 3x3 (+ folded BatchNorm bias, activation).  w is fp32 [9][C] tap-major.
__global__ void dw3x3_kernel(const __nv_bfloat16 *__restrict__ x, const float *__restrict__ w,
                             const float *__restrict__ b, __nv_bfloat16 *__restrict__ y, int N, int C, int H, int W,
                             int P, int Q, int stride, int pad, int act) {
    int C8 = C >> 3;
    long long total = (long long)N * P * Q * C8;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        int c0 = (int)(i % C8) * 8;
        long long t = i / C8;
        int q = (int)(t % Q); t /= Q;
        int p = (int)(t % P);
        int n = (int)(t / P);
        f8 acc;
        const float4 b0 = *reinterpret_cast<const float4 *>(b + c0), b1 = *reinterpret_cast<const float4 *>(b + c0 + 4);
        acc.v[0] = b0.x; acc.v[1] = b0.y; acc.v[2] = b0.z; acc.v[3] = b0.w;
        acc.v[4] = b1.x; acc.v[5] = b1.y; acc.v[6] = b1.z; acc.v[7] = b1.w;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            int ih = p * stride - pad + r;
            if (ih < 0 || ih >= H) continue;
#pragma unroll
            for (int s = 0; s < 3; ++s) {
                int iw = q * stride - pad + s;
                if (iw < 0 || iw >= W) continue;
                uint4 u = *reinterpret_cast<const uint4 *>(x + (((size_t)n * H + ih) * W + iw) * C + c0);
                f8 xv = unpack8(u);
                const float *wt = w + (size_t)(r * 3 + s) * C + c0;
                const float4 w0 = *reinterpret_cast<const float4 *>(wt), w1 = *reinterpret_cast<const float4 *>(wt + 4);
                acc.v[0] = fmaf(xv.v[0], w0.x, acc.v[0]); acc.v[1] = fmaf(xv.v[1], w0.y, acc.v[1]);
                acc.v[2] = fmaf(xv.v[2], w0.z, acc.v[2]); acc.v[3] = fmaf(xv.v[3], w0.w, acc.v[3]);
                acc.v[4] = fmaf(xv.v[4], w1.x, acc.v[4]); acc.v[5] = fmaf(xv.v[5], w1.y, acc.v[5]);
                acc.v[6] = fmaf(xv.v[6], w1.z, acc.v[6]); acc.v[7] = fmaf(xv.v[7], w1.w, acc.v[7]);
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) acc.v[j] = apply_act(acc.v[j], act);
        *reinterpret_cast<uint4 *>(y + (((size_t)n * P + p) * Q + q) * C + c0) = pack8(acc);
    }
}

// Max (kind 0) / average (kind 1) pooling.
__global__ void pool_kernel(const __nv_bfloat16 *__restrict__ x, __nv_bfloat16 *__restrict__ y, int N, int C, int H,
                            int W, int P, int Q, int k, int stride, int pad, int kind) {
    int C8 = C >> 3;
    long long total = (long long)N * P * Q * C8;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        int c0 = (int)(i % C8) * 8;
        long long t = i / C8;
        int q = (int)(t % Q); t /= Q;
        int p = (int)(t % P);
        int n = (int)(t / P);
        f8 m, sum;
#pragma unroll
        for (int j = 0; j < 8; ++j) { m.v[j] = -INFINITY; sum.v[j] = 0.0f; }
        int cnt = 0;
        for (int r = 0; r < k; ++r) {
            int ih = p * stride - pad + r;
            if (ih < 0 || ih >= H) continue;
            for (int s = 0; s < k; ++s) {
                int iw = q * stride - pad + s;
                if (iw < 0 || iw >= W) continue;
                f8 xv = unpack8(*reinterpret_cast<const uint4 *>(x + (((size_t)n * H + ih) * W + iw) * C + c0));
#pragma unroll
                for (int j = 0; j < 8; ++j) { m.v[j] = fmaxf(m.v[j], xv.v[j]); sum.v[j] += xv.v[j]; }
                ++cnt;
            }
        }
        if (kind == 1) {
#pragma unroll
            for (int j = 0; j < 8; ++j) m.v[j] = cnt ? sum.v[j] / (float)cnt : 0.0f;
        }
        *reinterpret_cast<uint4 *>(y + (((size_t)n * P + p) * Q + q) * C + c0) = pack8(m);
    }
}

// Global average over H*W: one thread per (image, 8 channels), rows summed in ascending order.
__global__ void gap_kernel(const __nv_bfloat16 *__restrict__ x, void *__restrict__ y, int N, int C, int HW, int out_f32) {
    int C8 = C >> 3;
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * C8) return;
    int c0 = (i % C8) * 8, n = i / C8;
    f8 sum;
#pragma unroll
    for (int j = 0; j < 8; ++j) sum.v[j] = 0.0f;
    for (int r = 0; r < HW; ++r) {
        f8 xv = unpack8(*reinterpret_cast<const uint4 *>(x + ((size_t)n * HW + r) * C + c0));
#pragma unroll
        for (int j = 0; j < 8; ++j) sum.v[j] += xv.v[j];
    }
    float inv = 1.0f / (float)HW;
#pragma unroll
    for (int j = 0; j < 8; ++j) sum.v[j] *= inv;
    if (out_f32) {
        float *o = reinterpret_cast<float *>(y) + (size_t)n * C + c0;
#pragma unroll
        for (int j = 0; j < 8; ++j) o[j] = sum.v[j];
    } else {
        *reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(y) + (size_t)n * C + c0) = pack8(sum);
    }
}

// 3x3 convolution of an NCHW image with at most 4 channels (the first layer of the bf16 graphs) on the CUDA cores:
// with K = 27 the MMA's 64-wide K block is mostly padding and building that block costs more than the product.
// A CTA takes 8 x 32 output pixels: the input window goes to shared memory as fp32 (zero outside the image = the
// padding), the weights [tap row][tap column][channel][Cout] and the bias too.  A thread owns 4 adjacent pixels of a
// row for 8 output channels: per tap row and input channel it reads the 4 pixels' window once and feeds 3 x 4 x 8
// multiply-adds; taps are added in the order (row, channel, column), fixed.  Output: NHWC bf16 (bias, activation).
template <typename TIn>
__global__ void __launch_bounds__(256)
stem3x3_kernel(const TIn *__restrict__ x, const float *__restrict__ w, const float *__restrict__ bias, __nv_bfloat16 *__restrict__ y,
               int N, int C, int H, int W, int K, int P, int Q, int stride, int pad, int act) {
    constexpr int TH = 8, TW = 32;
    extern __shared__ float stem_sm[];
    const int ih = (TH - 1) * stride + 3, iw = (TW - 1) * stride + 3, iwp = iw | 1;       // odd pitch: fewer bank conflicts
    float *win = stem_sm;                                  // [C][ih][iwp]
    float *ws = win + ((C * ih * iwp + 3) & ~3);           // [3][3][C][K], 16-byte aligned
    float *bs = ws + 9 * C * K;                            // [K]
    const int tiles_x = (Q + TW - 1) / TW, tiles_y = (P + TH - 1) / TH;
    const int t = blockIdx.x % (tiles_x * tiles_y), n = blockIdx.x / (tiles_x * tiles_y);
    const int ty = t / tiles_x, tx = t - ty * tiles_x;
    const int y0 = ty * TH * stride - pad, x0 = tx * TW * stride - pad;
    // the next kernel of the stream may be scheduled as soon as every CTA of this one has started
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int i = threadIdx.x; i < 9 * C * K; i += 256) ws[i] = w[i];
    for (int i = threadIdx.x; i < K; i += 256) bs[i] = bias[i];
    // window rows: a warp takes a (channel, row) pair at a time, its lanes three columns each: independent loads, no
    // division in the loop
    {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        for (int cr = warp; cr < C * ih; cr += 8) {
            const int c = cr / ih, yy = cr - c * ih, gy = y0 + yy;
            const bool row_in = gy >= 0 && gy < H;
            const TIn *src = x + (((size_t)n * C + c) * H + (row_in ? gy : 0)) * W;
            float v[3];
#pragma unroll
            for (int e = 0; e < 3; ++e) {
                const int xx = lane + 32 * e, gx = x0 + xx;
                v[e] = (row_in && xx < iw && gx >= 0 && gx < W) ? (float)src[gx] : 0.0f;
            }
#pragma unroll
            for (int e = 0; e < 3; ++e) {
                const int xx = lane + 32 * e;
                if (xx < iw) win[cr * iwp + xx] = v[e];
            }
        }
    }
    __syncthreads();
    const int K8 = K >> 3;
    const float lo = act >= 1 ? 0.0f : -INFINITY, hi = act == 2 ? 6.0f : INFINITY;
    for (int u = threadIdx.x; u < TH * (TW / 4) * K8; u += 256) {
        const int cg = u % K8, pg = u / K8, py = pg / (TW / 4), px = (pg - py * (TW / 4)) * 4;
        float2 acc[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int o = 0; o < 4; ++o) acc[j][o] = make_float2(bs[cg * 8 + 2 * o], bs[cg * 8 + 2 * o + 1]);
        for (int r = 0; r < 3; ++r)
            for (int c = 0; c < C; ++c) {
                const float *row = win + (c * ih + py * stride + r) * iwp + px * stride;
                float v[9];
#pragma unroll
                for (int e = 0; e < 9; ++e) v[e] = e < 3 * stride + 3 ? row[e] : 0.0f;      // (stride 1 uses 6, stride 2 uses 9)
#pragma unroll
                for (int s = 0; s < 3; ++s) {
                    const float4 w0 = *reinterpret_cast<const float4 *>(ws + ((r * 3 + s) * C + c) * K + cg * 8);
                    const float4 w1 = *reinterpret_cast<const float4 *>(ws + ((r * 3 + s) * C + c) * K + cg * 8 + 4);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float in = stride == 1 ? v[j + s] : v[2 * j + s];
                        const float2 in2 = make_float2(in, in);
                        acc[j][0] = __ffma2_rn(in2, make_float2(w0.x, w0.y), acc[j][0]);
                        acc[j][1] = __ffma2_rn(in2, make_float2(w0.z, w0.w), acc[j][1]);
                        acc[j][2] = __ffma2_rn(in2, make_float2(w1.x, w1.y), acc[j][2]);
                        acc[j][3] = __ffma2_rn(in2, make_float2(w1.z, w1.w), acc[j][3]);
                    }
                }
            }
        const int oy = ty * TH + py;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int ox = tx * TW + px + j;
            if (oy >= P || ox >= Q) continue;
            f8 o;
#pragma unroll
            for (int e = 0; e < 4; ++e) { o.v[2 * e] = fminf(fmaxf(acc[j][e].x, lo), hi); o.v[2 * e + 1] = fminf(fmaxf(acc[j][e].y, lo), hi); }
            *reinterpret_cast<uint4 *>(y + (((size_t)n * P + oy) * Q + ox) * K + cg * 8) = pack8(o);
        }
    }
}

// Fully connected layer (Eq. 1 of the Xenos paper: out = W x + b) for batches of at most 32 vectors, on the CUDA
// cores: with so few rows a 128-row MMA tile is three quarters empty and the layer is a single pass over the weight
// matrix.  The CTA stages the input vectors [N][C] in shared memory; a warp takes one output feature at a time: its
// lanes read the feature's weight row 16 bytes at a time (each weight leaves L2 once per CTA that needs it, once
// from HBM), multiply it with all N vectors, and the 32 lanes' partial sums are added by butterfly shuffles (a fixed
// order).  w is the packed [K padded][ldw] bf16 matrix of the implicit GEMM; bias, activation and output as there.
__global__ void __launch_bounds__(256)
fc_small_kernel(const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ w, const float *__restrict__ bias,
                void *__restrict__ y, int N, int C, int ldw, int K, int act, int out_f32, int out_ctot, int out_coff) {
    extern __shared__ uint4 fc_xs[];                       // [N][C / 8] chunks of 8 channels
    const int C8 = C >> 3;
    for (int i = threadIdx.x; i < N * C8; i += blockDim.x) fc_xs[i] = reinterpret_cast<const uint4 *>(x)[i];
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const float lo = act >= 1 ? 0.0f : -INFINITY, hi = act == 2 ? 6.0f : INFINITY;
    for (int o = blockIdx.x * nwarps + warp; o < K; o += gridDim.x * nwarps) {
        float acc[32];
#pragma unroll
        for (int n = 0; n < 32; ++n) acc[n] = 0.0f;
        const uint4 *wrow = reinterpret_cast<const uint4 *>(w + (size_t)o * ldw);
        for (int ch = lane; ch < C8; ch += 32) {
            const f8 wv = unpack8(__ldg(wrow + ch));
#pragma unroll
            for (int n = 0; n < 32; ++n) {
                if (n >= N) break;
                const f8 xv = unpack8(fc_xs[n * C8 + ch]);
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[n] = fmaf(wv.v[j], xv.v[j], acc[n]);
            }
        }
#pragma unroll
        for (int n = 0; n < 32; ++n) {
            if (n >= N) break;
            float v = acc[n];
#pragma unroll
            for (int s = 16; s >= 1; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
            acc[n] = v;
        }
        // lane n stores image n
        float mine = 0.0f;
#pragma unroll
        for (int n = 0; n < 32; ++n) if (n == lane) mine = acc[n];
        if (lane < N) {
            const float r = fminf(fmaxf(mine + bias[o], lo), hi);
            const size_t oi = (size_t)lane * out_ctot + out_coff + o;
            if (out_f32) reinterpret_cast<float *>(y)[oi] = r;
            else reinterpret_cast<__nv_bfloat16 *>(y)[oi] = __float2bfloat16_rn(r);
        }
    }
}

__global__ void add_kernel(const __nv_bfloat16 *__restrict__ a, const __nv_bfloat16 *__restrict__ b,
                           __nv_bfloat16 *__restrict__ y, long long n8, int act) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n8; i += (long long)gridDim.x * blockDim.x) {
        f8 av = unpack8(reinterpret_cast<const uint4 *>(a)[i]);
        f8 bv = unpack8(reinterpret_cast<const uint4 *>(b)[i]);
#pragma unroll
        for (int j = 0; j < 8; ++j) av.v[j] = apply_act(av.v[j] + bv.v[j], act);
        reinterpret_cast<uint4 *>(y)[i] = pack8(av);
    }
}

// x.mul (c == nullptr): a * b; x.mac: a * b + c.  The product is rounded to fp32 before the sum (no fused
// multiply-add), as the operator-at-a-time definition has it.
__global__ void mulmac_kernel(const __nv_bfloat16 *__restrict__ a, const __nv_bfloat16 *__restrict__ b,
                              const __nv_bfloat16 *__restrict__ c, __nv_bfloat16 *__restrict__ y, long long n8) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n8; i += (long long)gridDim.x * blockDim.x) {
        f8 av = unpack8(reinterpret_cast<const uint4 *>(a)[i]);
        const f8 bv = unpack8(reinterpret_cast<const uint4 *>(b)[i]);
#pragma unroll
        for (int j = 0; j < 8; ++j) av.v[j] = __fmul_rn(av.v[j], bv.v[j]);
        if (c) {
            const f8 cv = unpack8(reinterpret_cast<const uint4 *>(c)[i]);
#pragma unroll
            for (int j = 0; j < 8; ++j) av.v[j] = __fadd_rn(av.v[j], cv.v[j]);
        }
        reinterpret_cast<uint4 *>(y)[i] = pack8(av);
    }
}

// x.transpose: per image x [R][Cc] -> y [Cc][R], through a padded 32 x 32 tile so that reads and writes are coalesced.
template <typename T>
__global__ void transpose_kernel(const T *__restrict__ x, T *__restrict__ y, int R, int Cc) {
    __shared__ T tile[32][33];
    const size_t img = (size_t)blockIdx.z * R * Cc;
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    for (int j = threadIdx.y; j < 32; j += blockDim.y) {
        const int r = r0 + j, c = c0 + threadIdx.x;
        if (r < R && c < Cc) tile[j][threadIdx.x] = x[img + (size_t)r * Cc + c];
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += blockDim.y) {
        const int c = c0 + j, r = r0 + threadIdx.x;
        if (r < R && c < Cc) y[img + (size_t)c * R + r] = tile[threadIdx.x][j];
    }
}

// x.split, one part: y [pixels][Ci] = x [pixels][Ctot] at channel offset coff.
__global__ void slice_kernel(const __nv_bfloat16 *__restrict__ x, __nv_bfloat16 *__restrict__ y,
                             long long pixels, int Ci, int Ctot, int coff) {
    int C8 = Ci >> 3;
    long long total = pixels * C8;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        long long px = i / C8;
        int c0 = (int)(i % C8) * 8;
        *reinterpret_cast<uint4 *>(y + px * Ci + c0) = *reinterpret_cast<const uint4 *>(x + px * Ctot + coff + c0);
    }
}

// One concat input: x [pixels][Ci] -> y [pixels][Ctot] at channel offset coff.
__global__ void concat_part_kernel(const __nv_bfloat16 *__restrict__ x, __nv_bfloat16 *__restrict__ y,
                                   long long pixels, int Ci, int Ctot, int coff) {
    int C8 = Ci >> 3;
    long long total = pixels * C8;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        long long px = i / C8;
        int c0 = (int)(i % C8) * 8;
        *reinterpret_cast<uint4 *>(y + px * Ctot + coff + c0) = *reinterpret_cast<const uint4 *>(x + px * Ci + c0);
    }
}

}  // namespace xk
