// Two linked convolutions in one kernel (Table 1 of the Xenos paper, row ConvX -> ConvY: Conv k x k -> Conv 1x1,
// Conv 3x3 -> Conv 3x3; with the shortcut row's identity branch added in the second epilogue).
//
// The first convolution's result never leaves the SM.  Per tile:
//   GEMM 1   activation boxes by TMA (the tile's patch shifted by the tap, zero fill = padding) x weight tiles
//            -> accumulator 1 in tensor memory (all Cmid <= 256 output channels of the tile's pixels)
//   middle   epilogue warps: bias, activation, bf16, stored in shared memory IN THE OPERAND LAYOUT the second
//            convolution reads (Section 4.1: the producer writes in the order the consumer reads): 64-channel
//            blocks of 128-byte rows, 128-byte swizzle; pixels outside the feature map are zeros (the second
//            convolution's padding)
//   GEMM 2   its activation operand IS that buffer: for tap (dy, dx) the operand is the same rows shifted by
//            dy * pitch + dx (the consumer's rows use the producer patch's pitch, so a tap is a constant row
//            offset), weight tiles by TMA -> accumulator 2, one output-channel tile after the other
//   final    bias, activation, identity shortcut, activation, store
// A 3x3 consumer needs the producer's patch with a one-pixel frame: the producer tile is rh1 x rw1 <= 128 pixels,
// the consumer's rh1 - 2 x rw1 - 2 of them (the frame is recomputed by neighbouring tiles: the halo of Section 4.1).
// Every wait is bounded; on expiry the role records XENOS_E_TIMEOUT and leaves through the common exit.
#pragma once

#include "gemm_tc.cuh"

namespace xk {

constexpr int kC2Threads = 64 + 256;            // TMA warp, MMA warp, eight epilogue warps
constexpr int kC2MidRows = kTileM + 64;         // rows of a middle block: the tile plus the largest tap offset
constexpr int kC2MidBlock = kC2MidRows * 128;   // bytes of one 64-channel block of the middle buffer

struct Chain2Params {
    const float *bias1, *bias2;
    const __nv_bfloat16 *skip;
    __nv_bfloat16 *out;
    unsigned int *status;
    int batch, P, Q;
    int k1, pad1, cpb1, kblocks1;       // first convolution: window, padding, 64-channel blocks per tap, K blocks
    int k2, cpb2, kblocks2;             // second convolution (stride 1, padding (k2 - 1) / 2)
    int n1pad, N2, tile_n2, n2_tiles;
    int rh1, rw1, halo, rh2, rw2, tiles_y, tiles_x, m_tiles;
    int stages, stage_bytes, a_box_bytes;
    int off_mid, off_bar;
    int act1, act2, act3, out_ctot, out_coff, skip_ctot;
    uint32_t idesc1, idesc2;
    int launch_id;
};

__device__ __forceinline__ unsigned c2_timeout_word(const Chain2Params &g, int role) {
    return kStatusTimeout | ((unsigned)role << 8) | (((unsigned)g.launch_id & 0xfffu) << 12);
}

__global__ void __launch_bounds__(kC2Threads, 1)
chain2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB1,
              const __grid_constant__ CUtensorMap tmB2, const Chain2Params g) {
    extern __shared__ uint8_t smem_raw[];
    pdl_launch_dependents();
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t sbase = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (sbase - raw);
    const uint32_t bar_base = sbase + g.off_bar;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
    const uint32_t acc1f_bar = bar_base + 8u * (2 * kMaxStages), acc1e_bar = acc1f_bar + 8u, midf_bar = acc1f_bar + 16u,
                   midfree_bar = acc1f_bar + 24u, acc2f_bar = acc1f_bar + 32u, acc2e_bar = acc1f_bar + 40u;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(sm + g.off_bar + 8 * (2 * kMaxStages + 6));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t mid = sbase + g.off_mid;
    const int epi_warps = (kC2Threads - 64) / 32;

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(acc1f_bar, 1); mbar_init(acc1e_bar, epi_warps); mbar_init(midf_bar, epi_warps);
        mbar_init(midfree_bar, 1); mbar_init(acc2f_bar, 1); mbar_init(acc2e_bar, epi_warps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB1) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB2) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // rows behind the tile (reached only through tap offsets, by consumer rows that are never stored) start as zeros
    for (int idx = threadIdx.x; idx < g.cpb2 * kC2MidRows * 8; idx += kC2Threads)
        st_shared16(mid + (uint32_t)idx * 16u, make_uint4(0u, 0u, 0u, 0u));
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t acc1 = tmem_base, acc2 = tmem_base + 256u;
    bool ok = true;
    if (warp != 1) pdl_wait();
    const int per_img = g.tiles_y * g.tiles_x;

    if (warp == 0) {
        if (lane == 0) {
            Ring st = {0, 0u};
            for (int ti = blockIdx.x; ti < g.m_tiles && ok; ti += gridDim.x) {
                const int n = ti / per_img, t = ti - n * per_img, ty = t / g.tiles_x, tx = t - ty * g.tiles_x;
                const int y0 = ty * g.rh2 - g.halo - g.pad1, x0 = tx * g.rw2 - g.halo - g.pad1;
                int tap_r = 0, tap_s = 0, cb = 0;
                for (int kb = 0; kb < g.kblocks1 && ok; ++kb) {
                    ok = mbar_wait(empty_bar(st.s), st.ph ^ 1u);
                    if (!ok) break;
                    const uint32_t a = sbase + st.s * g.stage_bytes;
                    mbar_arrive_expect_tx(full_bar(st.s), (uint32_t)(g.a_box_bytes + g.n1pad * 128));
                    tma_load_4d(a, &tmA, cb * kTileK, x0 + tap_s, y0 + tap_r, n, full_bar(st.s));
                    tma_load_2d(a + kABytes, &tmB1, kb * kTileK, 0, full_bar(st.s));
                    st.next(g.stages);
                    if (++cb == g.cpb1) { cb = 0; if (++tap_s == g.k1) { tap_s = 0; ++tap_r; } }
                }
                for (int n2 = 0; n2 < g.n2_tiles && ok; ++n2)
                    for (int kb = 0; kb < g.kblocks2 && ok; ++kb) {
                        ok = mbar_wait(empty_bar(st.s), st.ph ^ 1u);
                        if (!ok) break;
                        mbar_arrive_expect_tx(full_bar(st.s), (uint32_t)g.tile_n2 * 128u);
                        tma_load_2d(sbase + st.s * g.stage_bytes + kABytes, &tmB2, kb * kTileK, n2 * g.tile_n2, full_bar(st.s));
                        st.next(g.stages);
                    }
            }
            if (!ok) atomicCAS(g.status, 0u, c2_timeout_word(g, 1));
        }
    } else if (warp == 1) {
        if (lane == 0) {
            Ring st = {0, 0u};
            int i = 0, j = 0;
            for (int ti = blockIdx.x; ti < g.m_tiles && ok; ti += gridDim.x, ++i) {
                ok = mbar_wait(acc1e_bar, (uint32_t)(i & 1) ^ 1u);          // the middle stage has read accumulator 1
                if (!ok) break;
                tc_fence_after();
                for (int kb = 0; kb < g.kblocks1 && ok; ++kb) {
                    const int s = st.s;
                    ok = mbar_wait(full_bar(s), st.ph);
                    if (!ok) break;
                    st.next(g.stages);
                    tc_fence_after();
                    const uint32_t a = sbase + s * g.stage_bytes, bb = a + kABytes;
#pragma unroll
                    for (int k4 = 0; k4 < kTileK / 16; ++k4)
                        umma_bf16(acc1, umma_desc_sw128(a + k4 * 32), umma_desc_sw128(bb + k4 * 32), g.idesc1, (kb > 0 || k4 > 0) ? 1u : 0u);
                    umma_commit(empty_bar(s));
                }
                if (!ok) break;
                umma_commit(acc1f_bar);
                ok = mbar_wait(midf_bar, (uint32_t)(i & 1));                // the middle tile is in shared memory
                if (!ok) break;
                fence_proxy_async();
                tc_fence_after();
                for (int n2 = 0; n2 < g.n2_tiles && ok; ++n2, ++j) {
                    ok = mbar_wait(acc2e_bar, (uint32_t)(j & 1) ^ 1u);      // the final epilogue has read accumulator 2
                    if (!ok) break;
                    tc_fence_after();
                    int dy = 0, dx = 0, cb = 0;
                    for (int kb = 0; kb < g.kblocks2 && ok; ++kb) {
                        const int s = st.s;
                        ok = mbar_wait(full_bar(s), st.ph);
                        if (!ok) break;
                        st.next(g.stages);
                        tc_fence_after();
                        // the consumer's operand for this tap: the middle rows, shifted by the tap's constant offset
                        const uint32_t a = mid + (uint32_t)cb * kC2MidBlock + (uint32_t)(dy * g.rw1 + dx) * 128u;
                        const uint32_t bb = sbase + s * g.stage_bytes + kABytes;
#pragma unroll
                        for (int k4 = 0; k4 < kTileK / 16; ++k4)
                            umma_bf16(acc2, umma_desc_sw128(a + k4 * 32), umma_desc_sw128(bb + k4 * 32), g.idesc2, (kb > 0 || k4 > 0) ? 1u : 0u);
                        umma_commit(empty_bar(s));
                        if (++cb == g.cpb2) { cb = 0; if (++dx == g.k2) { dx = 0; ++dy; } }
                    }
                    if (ok) umma_commit(acc2f_bar);
                }
                if (ok) umma_commit(midfree_bar);                           // every product that reads the middle tile is done
            }
            if (!ok) atomicCAS(g.status, 0u, c2_timeout_word(g, 2));
        }
    } else {
        // ---- epilogue warps: two per quarter of the accumulator's lanes, alternate 32-column chunks ----
        const int quarter = warp & 3, half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
        const float lo1 = act_lo(g.act1), hi1 = act_hi(g.act1), lo2 = act_lo(g.act2), hi2 = act_hi(g.act2);
        const float lo3 = act_lo(g.act3), hi3 = act_hi(g.act3);
        const int ry = row / g.rw1, rx = row - ry * g.rw1;
        int i = 0, j = 0;
        for (int ti = blockIdx.x; ti < g.m_tiles && ok; ti += gridDim.x, ++i) {
            const int n = ti / per_img, t = ti - n * per_img, ty = t / g.tiles_x, tx = t - ty * g.tiles_x;
            // producer pixel of this row (frame included) and whether it lies in the feature map
            const int py = ty * g.rh2 - g.halo + ry, px = tx * g.rw2 - g.halo + rx;
            const bool inside = row < g.rh1 * g.rw1 && py >= 0 && py < g.P && px >= 0 && px < g.Q;
            ok = mbar_wait_warp(acc1f_bar, (uint32_t)(i & 1), lane) && mbar_wait_warp(midfree_bar, (uint32_t)(i & 1) ^ 1u, lane);
            if (!ok) break;
            tc_fence_after();
            for (int c32 = half; c32 * 32 < g.n1pad; c32 += 2) {
                float v[32];
                if (c32 * 32 + 32 <= g.n1pad) tmem_ld32(acc1 + lane_off + c32 * 32, v);
                else { tmem_ld16(acc1 + lane_off + c32 * 32, v); for (int q = 16; q < 32; ++q) v[q] = 0.0f; }
#pragma unroll
                for (int q8 = 0; q8 < 32; q8 += 8) {
                    const int col = c32 * 32 + q8;
                    if (col >= g.n1pad) break;
                    const float4 b0 = __ldg(reinterpret_cast<const float4 *>(g.bias1 + col)), b1 = __ldg(reinterpret_cast<const float4 *>(g.bias1 + col + 4));
                    f8 o;
                    o.v[0] = v[q8] + b0.x; o.v[1] = v[q8 + 1] + b0.y; o.v[2] = v[q8 + 2] + b0.z; o.v[3] = v[q8 + 3] + b0.w;
                    o.v[4] = v[q8 + 4] + b1.x; o.v[5] = v[q8 + 5] + b1.y; o.v[6] = v[q8 + 6] + b1.z; o.v[7] = v[q8 + 7] + b1.w;
#pragma unroll
                    for (int c = 0; c < 8; ++c) o.v[c] = inside ? fminf(fmaxf(o.v[c], lo1), hi1) : 0.0f;
                    st_shared16(a_chunk_addr(mid + (uint32_t)(col >> 6) * kC2MidBlock, row, (col & 63) >> 3), pack8(o));
                }
            }
            tc_fence_before();
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) { mbar_arrive(acc1e_bar); mbar_arrive(midf_bar); }
            // ---- final epilogue of every output-channel tile ----
            const int cy = ry, cx = rx;                                 // consumer row: same pitch, no frame
            const int oy = ty * g.rh2 + cy, ox = tx * g.rw2 + cx;
            const bool valid = cy < g.rh2 && cx < g.rw2 && oy < g.P && ox < g.Q && n < g.batch;
            const size_t pix = ((size_t)n * g.P + oy) * g.Q + ox;
            for (int n2 = 0; n2 < g.n2_tiles && ok; ++n2, ++j) {
                const int n0 = n2 * g.tile_n2;
                // the shortcut's values for this warp's first chunk are asked for before the accumulator is ready
                uint4 sk[4];
                auto load_skip = [&](int c32) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int col = n0 + c32 * 32 + q * 8;
                        sk[q] = (g.skip && valid && col + 8 <= g.N2) ? __ldg(reinterpret_cast<const uint4 *>(g.skip + pix * g.skip_ctot + col)) : make_uint4(0u, 0u, 0u, 0u);
                    }
                };
                load_skip(half);
                ok = mbar_wait_warp(acc2f_bar, (uint32_t)(j & 1), lane);
                if (!ok) break;
                tc_fence_after();
                for (int c32 = half; c32 * 32 < g.tile_n2; c32 += 2) {
                    float v[32];
                    if (c32 * 32 + 32 <= g.tile_n2) tmem_ld32(acc2 + lane_off + c32 * 32, v);
                    else { tmem_ld16(acc2 + lane_off + c32 * 32, v); for (int q = 16; q < 32; ++q) v[q] = 0.0f; }
                    if ((c32 + 2) * 32 >= g.tile_n2) {
                        // this warp's last read of accumulator 2
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(acc2e_bar);
                    }
                    uint4 skc[4] = {sk[0], sk[1], sk[2], sk[3]};
                    if ((c32 + 2) * 32 < g.tile_n2) load_skip(c32 + 2);       // next chunk's shortcut values in flight
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int col = n0 + c32 * 32 + q * 8;
                        if (c32 * 32 + q * 8 >= g.tile_n2 || col + 8 > g.N2 || !valid) continue;
                        const float4 b0 = __ldg(reinterpret_cast<const float4 *>(g.bias2 + col)), b1 = __ldg(reinterpret_cast<const float4 *>(g.bias2 + col + 4));
                        f8 o;
                        o.v[0] = v[q * 8] + b0.x; o.v[1] = v[q * 8 + 1] + b0.y; o.v[2] = v[q * 8 + 2] + b0.z; o.v[3] = v[q * 8 + 3] + b0.w;
                        o.v[4] = v[q * 8 + 4] + b1.x; o.v[5] = v[q * 8 + 5] + b1.y; o.v[6] = v[q * 8 + 6] + b1.z; o.v[7] = v[q * 8 + 7] + b1.w;
#pragma unroll
                        for (int c = 0; c < 8; ++c) o.v[c] = fminf(fmaxf(o.v[c], lo2), hi2);
                        if (g.skip) {
                            const f8 sv = unpack8(skc[q]);
#pragma unroll
                            for (int c = 0; c < 8; ++c) o.v[c] += sv.v[c];
                        }
#pragma unroll
                        for (int c = 0; c < 8; ++c) o.v[c] = fminf(fmaxf(o.v[c], lo3), hi3);
                        *reinterpret_cast<uint4 *>(g.out + pix * g.out_ctot + g.out_coff + col) = pack8(o);
                    }
                }
                if (half * 32 >= g.tile_n2 && lane == 0) mbar_arrive(acc2e_bar);      // a warp without a chunk in so narrow a tile
            }
        }
        if (!ok && lane == 0) atomicCAS(g.status, 0u, c2_timeout_word(g, 5));
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

}  // namespace xk
