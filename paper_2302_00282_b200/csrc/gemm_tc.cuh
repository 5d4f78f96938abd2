// Linked-chain implicit GEMM on the 5th-generation tensor cores (sm_100a).
//
// One CTA owns a 128-row tile of output pixels and a slice of <= 256 output channels
// (the operator split of Section 4.2: output channels first, then rows / columns).
//   warp 0      : TMA producer for the weight tile (cp.async.bulk.tensor, 128-byte swizzle)
//   warp 1      : allocates tensor memory, one lane issues tcgen05.mma (bf16 x bf16 -> fp32)
//   warps 2..5  : produce the activation operand straight into shared memory in the layout the
//                 tensor core reads (K-major, 128-byte swizzle) - the paper's "write in the
//                 order the next operator reads" (Section 4.1) - then run the epilogue
// The activation operand of one 64-wide K block comes from one of
//   gather : a k x k / strided / padded window of an NHWC bf16 tensor (16-byte cp.async, zero fill)
//   stem   : a k x k window of a small-channel NCHW image (scalar loads, converted to bf16)
//   dw     : a depthwise 3x3 + bias + activation computed on the fly (linked dw -> pw)
// and a second gather segment can append the K blocks of a shortcut 1x1 convolution, so the
// residual sum of a shortcut connection happens in the accumulator.
// Epilogues: bias, activation, identity-shortcut add, then a coalesced store at a channel
// offset (concat needs no kernel), a max pool over the tile's patch, or a global average.
//
// Every wait on an mbarrier is bounded; on expiry the CTA records XENOS_E_TIMEOUT in the status
// word and leaves through the common exit (tensor memory is always released).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels_bf16.cuh"

namespace xk {

enum { GA_NONE = 0, GA_GATHER = 1, GA_STEM = 2, GA_DW = 3 };
enum { GE_STORE = 0, GE_GAP = 1, GE_POOL = 2 };
enum { GM_FLAT = 0, GM_PATCH = 1 };

constexpr int kTileM = 128;
constexpr int kTileK = 64;
constexpr int kABytes = kTileM * kTileK * 2;    // 16 KB per stage
constexpr int kMaxStages = 6;
constexpr unsigned kStatusTimeout = 0x80000000u | 9u;
constexpr unsigned kStatusBounds = 0x80000000u | 10u;
constexpr int kSpinLimit = 1 << 22;             // try_wait polls before a wait gives up

struct GemmSeg {
    const void *src;
    const float *dw_w, *dw_b;
    int mode, C, H, W, k, stride, pad, kelems, kblocks, src_f32, dw_act;
};

struct GemmParams {
    GemmSeg seg[2];
    const float *bias;
    const __nv_bfloat16 *skip;
    void *out;
    unsigned int *status;
    int batch, P, Q, rpi;
    int map_mode, tile_rows, imgs_per_tile;
    int th, tw, rh, rw, tiles_y, tiles_x, pool_k, pool_stride, pool_pad, PP, PQ;
    int kblocks, stages, tile_n, n_tiles, N;
    int act, act2, epi, out_ctot, out_coff, out_f32, skip_ctot;
    uint32_t idesc;
};

// ---- PTX wrappers ------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for the phase with the given parity.  Returns false when it gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (int i = 0; i < kSpinLimit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void st_shared16(uint32_t dst, const uint4 &v) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 ld_shared16(uint32_t src) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(src));
    return v;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(x), "r"(y) : "memory");
}

// K-major operand tile with 128-byte swizzle: rows 128 bytes apart, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3ffffu) >> 4);          // start address, 16-byte units
    d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset: next 8-row group
    d |= (uint64_t)1 << 46;                            // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                            // 128-byte swizzle
    return d;
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// ---- row <-> pixel -----------------------------------------------------------------------------
struct RowPos { int valid, n, p, q; };

__device__ __forceinline__ RowPos map_row(const GemmParams &g, int mt, int r) {
    RowPos o;
    o.valid = 0; o.n = 0; o.p = 0; o.q = 0;
    if (g.map_mode == GM_FLAT) {
        long long m = (long long)mt * g.tile_rows + r;
        if (r < g.tile_rows && m < (long long)g.batch * g.rpi) {
            o.n = (int)(m / g.rpi);
            int rem = (int)(m - (long long)o.n * g.rpi);
            o.p = rem / g.Q; o.q = rem - o.p * g.Q;
            o.valid = 1;
        }
    } else {
        int per = g.tiles_y * g.tiles_x;
        o.n = mt / per;
        int t = mt - o.n * per;
        int ty = t / g.tiles_x, tx = t - ty * g.tiles_x;
        int dy = r / g.rw, dx = r - dy * g.rw;
        o.p = ty * g.th * g.pool_stride - g.pool_pad + dy;
        o.q = tx * g.tw * g.pool_stride - g.pool_pad + dx;
        o.valid = (r < g.rh * g.rw) && o.n < g.batch && o.p >= 0 && o.p < g.P && o.q >= 0 && o.q < g.Q;
    }
    return o;
}

// ---- A-operand producers: each of the 128 producer threads fills one row (128 bytes) of the stage
__device__ __forceinline__ uint32_t a_chunk_addr(uint32_t a_base, int row, int j) {
    return a_base + row * 128 + ((j ^ (row & 7)) << 4);
}

struct GatherState { int tap_r, tap_s, cc; };   // position of the next 8-channel chunk inside the segment

__device__ __forceinline__ void produce_gather(const GemmSeg &sg, GatherState &st, const RowPos &rp, uint32_t a_base, int row) {
    const __nv_bfloat16 *src = reinterpret_cast<const __nv_bfloat16 *>(sg.src);
    int C8 = sg.C >> 3;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const void *ptr = src;
        uint32_t bytes = 0;
        if (rp.valid && st.tap_r < sg.k) {
            int ih = rp.p * sg.stride - sg.pad + st.tap_r, iw = rp.q * sg.stride - sg.pad + st.tap_s;
            if (ih >= 0 && ih < sg.H && iw >= 0 && iw < sg.W) {
                ptr = src + (((size_t)rp.n * sg.H + ih) * sg.W + iw) * sg.C + st.cc * 8;
                bytes = 16;
            }
        }
        cp_async16(a_chunk_addr(a_base, row, j), ptr, bytes);
        if (st.tap_r < sg.k && ++st.cc == C8) {
            st.cc = 0;
            if (++st.tap_s == sg.k) { st.tap_s = 0; ++st.tap_r; }
        }
    }
}

// K order of the stem: element e = (r * k + s) * C + c of an NCHW image, fp32 or bf16.
__device__ __forceinline__ void produce_stem(const GemmSeg &sg, int kb_local, const RowPos &rp, uint32_t a_base, int row) {
    int e = kb_local * kTileK;
    int tap = e / sg.C, c = e - tap * sg.C;
    int r = tap / sg.k, s = tap - r * sg.k;
#pragma unroll 1
    for (int j = 0; j < 8; ++j) {
        f8 v;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float x = 0.0f;
            if (rp.valid && r < sg.k) {
                int ih = rp.p * sg.stride - sg.pad + r, iw = rp.q * sg.stride - sg.pad + s;
                if (ih >= 0 && ih < sg.H && iw >= 0 && iw < sg.W) {
                    size_t idx = (((size_t)rp.n * sg.C + c) * sg.H + ih) * sg.W + iw;
                    x = sg.src_f32 ? reinterpret_cast<const float *>(sg.src)[idx]
                                   : __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(sg.src)[idx]);
                }
            }
            v.v[i] = x;
            if (++c == sg.C) { c = 0; if (++s == sg.k) { s = 0; ++r; } }
        }
        st_shared16(a_chunk_addr(a_base, row, j), pack8(v));
    }
}

// Depthwise 3x3 + bias + activation for 64 channels of one output pixel, rounded to bf16.
__device__ __forceinline__ void produce_dw(const GemmSeg &sg, int kb_local, const RowPos &rp, uint32_t a_base, int row) {
    const __nv_bfloat16 *src = reinterpret_cast<const __nv_bfloat16 *>(sg.src);
#pragma unroll 1
    for (int j = 0; j < 8; ++j) {
        int c0 = kb_local * kTileK + j * 8;
        uint4 outv = make_uint4(0u, 0u, 0u, 0u);
        if (rp.valid && c0 < sg.C) {
            f8 acc;
            const float4 b0 = *reinterpret_cast<const float4 *>(sg.dw_b + c0), b1 = *reinterpret_cast<const float4 *>(sg.dw_b + c0 + 4);
            acc.v[0] = b0.x; acc.v[1] = b0.y; acc.v[2] = b0.z; acc.v[3] = b0.w;
            acc.v[4] = b1.x; acc.v[5] = b1.y; acc.v[6] = b1.z; acc.v[7] = b1.w;
#pragma unroll
            for (int r = 0; r < 3; ++r) {
                int ih = rp.p * sg.stride - sg.pad + r;
                if (ih < 0 || ih >= sg.H) continue;
#pragma unroll
                for (int s = 0; s < 3; ++s) {
                    int iw = rp.q * sg.stride - sg.pad + s;
                    if (iw < 0 || iw >= sg.W) continue;
                    f8 xv = unpack8(__ldg(reinterpret_cast<const uint4 *>(src + (((size_t)rp.n * sg.H + ih) * sg.W + iw) * sg.C + c0)));
                    const float *wt = sg.dw_w + (size_t)(r * 3 + s) * sg.C + c0;
                    const float4 w0 = __ldg(reinterpret_cast<const float4 *>(wt)), w1 = __ldg(reinterpret_cast<const float4 *>(wt + 4));
                    acc.v[0] = fmaf(xv.v[0], w0.x, acc.v[0]); acc.v[1] = fmaf(xv.v[1], w0.y, acc.v[1]);
                    acc.v[2] = fmaf(xv.v[2], w0.z, acc.v[2]); acc.v[3] = fmaf(xv.v[3], w0.w, acc.v[3]);
                    acc.v[4] = fmaf(xv.v[4], w1.x, acc.v[4]); acc.v[5] = fmaf(xv.v[5], w1.y, acc.v[5]);
                    acc.v[6] = fmaf(xv.v[6], w1.z, acc.v[6]); acc.v[7] = fmaf(xv.v[7], w1.w, acc.v[7]);
                }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) acc.v[i] = apply_act(acc.v[i], sg.dw_act);
            outv = pack8(acc);
        }
        st_shared16(a_chunk_addr(a_base, row, j), outv);
    }
}

// ---- the kernel --------------------------------------------------------------------------------
__global__ void __launch_bounds__(192) gemm_chain_kernel(const __grid_constant__ CUtensorMap tmB, const GemmParams g) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t sbase = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (sbase - raw);
    const int stage_bytes = kABytes + g.tile_n * 128;
    const uint32_t bar_base = sbase + g.stages * stage_bytes;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
    const uint32_t accum_bar = bar_base + 8u * (2 * kMaxStages);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(sm + g.stages * stage_bytes + 8 * (2 * kMaxStages + 1));
    int *abort_flag = reinterpret_cast<int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int mt = blockIdx.x / g.n_tiles, nt = blockIdx.x - mt * g.n_tiles;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < g.tile_n) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) { mbar_init(full_bar(s), 128 + 1); mbar_init(empty_bar(s), 1); }
        mbar_init(accum_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool ok = true;

    if (warp == 0) {
        // ---- weight tiles by TMA ----
        if (lane == 0) {
            for (int kb = 0; kb < g.kblocks && ok; ++kb) {
                int s = kb % g.stages;
                uint32_t ph = (kb / g.stages) & 1;
                ok = mbar_wait(empty_bar(s), ph ^ 1u);
                if (!ok) break;
                mbar_arrive_expect_tx(full_bar(s), (uint32_t)g.tile_n * 128u);
                tma_load_2d(sbase + s * stage_bytes + kABytes, &tmB, kb * kTileK, nt * g.tile_n, full_bar(s));
            }
            if (!ok) { atomicCAS(g.status, 0u, kStatusTimeout); atomicExch(abort_flag, 1); }
        }
    } else if (warp == 1) {
        // ---- MMA issue ----
        if (lane == 0) {
            for (int kb = 0; kb < g.kblocks && ok; ++kb) {
                int s = kb % g.stages;
                uint32_t ph = (kb / g.stages) & 1;
                ok = mbar_wait(full_bar(s), ph);
                if (!ok) break;
                tc_fence_after();
                uint32_t a = sbase + s * stage_bytes, b = a + kABytes;
#pragma unroll
                for (int k4 = 0; k4 < kTileK / 16; ++k4)
                    umma_bf16(tmem_base, umma_desc_sw128(a + k4 * 32), umma_desc_sw128(b + k4 * 32), g.idesc,
                              (kb > 0 || k4 > 0) ? 1u : 0u);
                umma_commit(empty_bar(s));
            }
            if (ok) umma_commit(accum_bar);
            else { atomicCAS(g.status, 0u, kStatusTimeout); atomicExch(abort_flag, 1); }
        }
    } else {
        // ---- activation operand, then epilogue ----
        const int row = (warp & 3) * 32 + lane;          // also the tensor-memory lane this thread reads
        const RowPos rp = map_row(g, mt, row);
        GatherState gs[2] = {{0, 0, 0}, {0, 0, 0}};
        const int lag = g.stages >= 3 ? 2 : 1;
        int pend = 0, pend_first = 0;
        auto retire_oldest = [&]() {
            fence_proxy_async();
            mbar_arrive(full_bar(pend_first % g.stages));
            ++pend_first; --pend;
        };
        for (int kb = 0; kb < g.kblocks && ok; ++kb) {
            int s = kb % g.stages;
            uint32_t ph = (kb / g.stages) & 1;
            ok = mbar_wait(empty_bar(s), ph ^ 1u);
            if (!ok) break;
            int si = kb < g.seg[0].kblocks ? 0 : 1;
            int kbl = kb - (si ? g.seg[0].kblocks : 0);
            const GemmSeg &sg = g.seg[si];
            uint32_t a_base = sbase + s * stage_bytes;
            if (sg.mode == GA_GATHER) {
                produce_gather(sg, gs[si], rp, a_base, row);
                cp_async_commit();
                ++pend;
                if (pend > lag) {
                    if (lag == 2) cp_async_wait<2>(); else cp_async_wait<1>();
                    retire_oldest();
                }
            } else {
                if (pend) { cp_async_wait<0>(); while (pend) retire_oldest(); }
                pend_first = kb + 1;
                if (sg.mode == GA_DW) produce_dw(sg, kbl, rp, a_base, row);
                else produce_stem(sg, kbl, rp, a_base, row);
                fence_proxy_async();
                mbar_arrive(full_bar(s));
            }
        }
        cp_async_wait<0>();
        if (ok) { while (pend) retire_oldest(); }
        else if (lane == 0) { atomicCAS(g.status, 0u, kStatusTimeout); atomicExch(abort_flag, 1); }

        // ---- epilogue ----
        if (ok) ok = mbar_wait(accum_bar, 0);
        ok = __all_sync(0xffffffffu, ok);     // warp-uniform from here on (tcgen05.ld is warp-collective)
        if (!ok && lane == 0) { atomicCAS(g.status, 0u, kStatusTimeout); atomicExch(abort_flag, 1); }
        tc_fence_after();
        const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const int n0 = nt * g.tile_n;
        const int nchunks = g.tile_n / 16;
        // staging area for the pool / global-average epilogues reuses the pipeline buffers: every
        // MMA has retired (accum barrier) so nothing reads or writes them any more
        const uint32_t stg = sbase;
        const int pool_pitch = g.tile_n * 2 + 16;
        for (int ch = 0; ch < nchunks; ++ch) {
            float v[16];
            if (ok) tmem_ld16(t_lane + ch * 16, v);
            else {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = 0.0f;
            }
            const int nc = n0 + ch * 16;
#pragma unroll
            for (int i = 0; i < 16; i += 4) {
                float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
                if (nc + i < g.N) b = __ldg(reinterpret_cast<const float4 *>(g.bias + nc + i));
                v[i] = apply_act(v[i] + b.x, g.act); v[i + 1] = apply_act(v[i + 1] + b.y, g.act);
                v[i + 2] = apply_act(v[i + 2] + b.z, g.act); v[i + 3] = apply_act(v[i + 3] + b.w, g.act);
            }
            // shortcut connection with an identity branch: the skip tile is read once, here
            const size_t pix = ((size_t)rp.n * g.P + rp.p) * g.Q + rp.q;
            if (g.skip && rp.valid) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (nc + h * 8 + 8 > g.N) break;
                    f8 sv = unpack8(__ldg(reinterpret_cast<const uint4 *>(g.skip + pix * g.skip_ctot + nc + h * 8)));
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[h * 8 + i] += sv.v[i];
                }
            }
            if (g.act2) {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = apply_act(v[i], g.act2);
            }
            if (g.epi == GE_STORE) {
                if (!rp.valid || !ok) continue;
                if (g.out_f32) {
                    float *o = reinterpret_cast<float *>(g.out) + pix * g.out_ctot + g.out_coff + nc;
#pragma unroll
                    for (int i = 0; i < 16; ++i) if (nc + i < g.N) o[i] = v[i];
                } else {
                    __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(g.out) + pix * g.out_ctot + g.out_coff + nc;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (nc + h * 8 + 8 > g.N) break;
                        f8 pv;
#pragma unroll
                        for (int i = 0; i < 8; ++i) pv.v[i] = v[h * 8 + i];
                        *reinterpret_cast<uint4 *>(o + h * 8) = pack8(pv);
                    }
                }
            } else if (g.epi == GE_POOL) {
                // rows outside the conv output never win a max
                f8 lo, hi;
#pragma unroll
                for (int i = 0; i < 8; ++i) { lo.v[i] = rp.valid ? v[i] : -INFINITY; hi.v[i] = rp.valid ? v[8 + i] : -INFINITY; }
                st_shared16(stg + row * pool_pitch + ch * 32, pack8(lo));
                st_shared16(stg + row * pool_pitch + ch * 32 + 16, pack8(hi));
            } else {
                // global average: 16 columns at a time through shared memory, rows summed in ascending order
                epi_bar();
                float *sf = reinterpret_cast<float *>(sm);
#pragma unroll
                for (int i = 0; i < 16; ++i) sf[row * 17 + i] = rp.valid ? v[i] : 0.0f;
                epi_bar();
                int t = threadIdx.x - 64;
                for (int item = t; item < g.imgs_per_tile * 16; item += 128) {
                    int img = item >> 4, c = item & 15;
                    int n = mt * g.imgs_per_tile + img;
                    if (n >= g.batch || nc + c >= g.N || !ok) continue;
                    float acc = 0.0f;
                    for (int r = 0; r < g.rpi; ++r) acc += sf[(img * g.rpi + r) * 17 + c];
                    acc /= (float)g.rpi;
                    size_t oi = (size_t)n * g.out_ctot + g.out_coff + nc + c;
                    if (g.out_f32) reinterpret_cast<float *>(g.out)[oi] = acc;
                    else reinterpret_cast<__nv_bfloat16 *>(g.out)[oi] = __float2bfloat16_rn(acc);
                }
            }
        }
        if (g.epi == GE_POOL) {
            epi_bar();
            int per = g.tiles_y * g.tiles_x;
            int n = mt / per, tt = mt - n * per;
            int ty = tt / g.tiles_x, tx = tt - ty * g.tiles_x;
            int c8n = g.tile_n / 8;
            int t = threadIdx.x - 64;
            for (int item = t; item < g.th * g.tw * c8n; item += 128) {
                int c8 = item % c8n, o = item / c8n;
                int oy = o / g.tw, ox = o - oy * g.tw;
                int gy = ty * g.th + oy, gx = tx * g.tw + ox;
                int col = n0 + c8 * 8;
                if (gy >= g.PP || gx >= g.PQ || col + 8 > g.N || n >= g.batch || !ok) continue;
                f8 m;
#pragma unroll
                for (int i = 0; i < 8; ++i) m.v[i] = -INFINITY;
                for (int dy = 0; dy < g.pool_k; ++dy)
                    for (int dx = 0; dx < g.pool_k; ++dx) {
                        int r = (oy * g.pool_stride + dy) * g.rw + ox * g.pool_stride + dx;
                        f8 xv = unpack8(ld_shared16(stg + r * pool_pitch + c8 * 16));
#pragma unroll
                        for (int i = 0; i < 8; ++i) m.v[i] = fmaxf(m.v[i], xv.v[i]);
                    }
                __nv_bfloat16 *o2 = reinterpret_cast<__nv_bfloat16 *>(g.out) +
                                    (((size_t)n * g.PP + gy) * g.PQ + gx) * g.out_ctot + g.out_coff + col;
                *reinterpret_cast<uint4 *>(o2) = pack8(m);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

}  // namespace xk
