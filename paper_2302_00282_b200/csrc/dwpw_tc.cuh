// Depthwise 3x3 -> pointwise 1x1 (Sections 2.2 and 4.1 of the Xenos paper: the depthwise result is produced in the
// layout the pointwise product reads and never leaves the SM), as a kernel of its own for the chains that store
// their tile.  It takes the same plan record and parameters as the depthwise mode of gemm_chain_kernel and differs
// in how the warps are used: there are no separate producer and epilogue warps.  Every worker warp runs the
// depthwise stencil of a tile's K blocks and then a share of the store epilogue of the previous tile, so that no
// warp waits for another role's stage, and all warps of a scheduler run the same loop.
//   warp 0   TMA: the tile's input window per 64-channel block (zero fill = padding), pointwise weight blocks
//   warp 1   MMA: acc[128 x tile_n] += A block x W block, two accumulators in tensor memory
//   workers  tile i + 1: stencil of every K block into the A|B ring; then tile i: bias, activation, bf16, store
// With kW = 16 the 512 worker threads each own 1 x 4 output pixels of 4 channels of a 64-channel block; with
// kW = 8 the 256 threads own 2 x 4 pixels (64-channel blocks) or 1 x 4 (narrower blocks).
// Every wait is bounded; on expiry the role records XENOS_E_TIMEOUT and the workers leave together.
#pragma once

#include "gemm_tc.cuh"

namespace xk {

template <int kW>
__global__ void __launch_bounds__(64 + 32 * kW, 1)
dwpw_kernel(const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmH, const GemmParams g) {
    constexpr int kWorkerThreads = 32 * kW;
    extern __shared__ uint8_t smem_raw[];
    pdl_launch_dependents();
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t sbase = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (sbase - raw);
    const int cols = g.n_acc * g.tile_n;                  // columns of a CTA's tile (n_acc = 2: both accumulators, 2 x 256)
    const int stage_bytes = kABytes + cols * 128;
    const uint32_t bar_base = sbase + g.off_bar;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
    auto accf_bar = [&](int b) { return bar_base + 8u * (2 * kMaxStages + b); };
    auto acce_bar = [&](int b) { return bar_base + 8u * (2 * kMaxStages + 2 + b); };
    auto hfull_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + 4 + s); };
    auto hempty_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + 4 + kMaxHaloStages + s); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(sm + g.off_bar + 8 * (2 * kMaxStages + 4 + 2 * kMaxHaloStages));
    volatile int *fail_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const uint32_t dww_bar = bar_base + 8u * (2 * kMaxStages + 4 + 2 * kMaxHaloStages + 3);      // the depthwise parameters have landed

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = g.m_tiles * g.n_tiles;
    const int dw_quads = g.halo_cb > 32 ? 16 : 8;
    const int dw_br = (g.halo_cb > 32 && kW == 8) ? 2 : 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) { mbar_init(full_bar(s), kW + 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), kW); }
        for (int s = 0; s < g.hstages; ++s) { mbar_init(hfull_bar(s), 1); mbar_init(hempty_bar(s), kW); }
        mbar_init(dww_bar, 1);
        *fail_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // depthwise tap weights [9][C] followed by the bias [C], fp32, once per CTA: two bulk copies that the workers wait
        // for before their first stencil (constants: no need to wait for the predecessor kernel)
        {
            const uint32_t C = (uint32_t)g.seg[0].C;
            mbar_arrive_expect_tx(dww_bar, 40u * C);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(sbase + g.off_dww), "l"(g.seg[0].dw_w), "r"(36u * C), "r"(dww_bar) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(sbase + g.off_dww + 36u * C), "l"(g.seg[0].dw_b), "r"(4u * C), "r"(dww_bar) : "memory");
        }
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmH) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)g.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool ok = true;
    if (warp != 1) pdl_wait();

    if (warp == 0) {
        if (lane == 0) {
            TileWalk w;
            w.init(g);
            Ring st = {0, 0u}, hr = {0, 0u};
            for (; w.ti < total_tiles && ok; w.next(g)) {
                const int hn = w.grp * g.ni;
                const int hy = (w.ty * g.step_y - g.off_y) * g.seg[0].stride - g.seg[0].pad;
                const int hx = (w.tx * g.step_x - g.off_x) * g.seg[0].stride - g.seg[0].pad;
                for (int kb = 0; kb < g.kblocks && ok; ++kb) {
                    ok = mbar_wait(hempty_bar(hr.s), hr.ph ^ 1u);
                    if (!ok) break;
                    mbar_arrive_expect_tx(hfull_bar(hr.s), (uint32_t)g.halo_bytes);
                    tma_load_4d(sbase + g.off_halo + hr.s * g.halo_stride, &tmH, kb * kTileK, hx, hy, hn, hfull_bar(hr.s));
                    hr.next(g.hstages);
                    ok = mbar_wait(empty_bar(st.s), st.ph ^ 1u);
                    if (!ok) break;
                    mbar_arrive_expect_tx(full_bar(st.s), (uint32_t)cols * 128u);
                    for (int h = 0; h < g.n_acc; ++h)
                        tma_load_2d(sbase + st.s * stage_bytes + kABytes + h * g.tile_n * 128, &tmB, kb * kTileK, (w.nt * g.n_acc + h) * g.tile_n, full_bar(st.s));
                    st.next(g.stages);
                }
            }
            if (!ok) atomicCAS(g.status, 0u, timeout_word(g, 1));
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int i = 0;
            Ring st = {0, 0u};
            for (int ti = blockIdx.x; ti < total_tiles && ok; ti += gridDim.x, ++i) {
                const int b = i & 1;
                ok = mbar_wait(acce_bar(b), ((i >> 1) & 1) ^ 1u);      // the workers have drained this accumulator
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + b * g.acc_stride;
                for (int kb = 0; kb < g.kblocks && ok; ++kb) {
                    const int s = st.s;
                    ok = mbar_wait(full_bar(s), st.ph);
                    if (!ok) break;
                    st.next(g.stages);
                    fence_proxy_async();
                    tc_fence_after();
                    const uint32_t a = sbase + s * stage_bytes, bb = a + kABytes;
                    for (int h = 0; h < g.n_acc; ++h)
#pragma unroll
                        for (int k4 = 0; k4 < kTileK / 16; ++k4)
                            umma_bf16(d_tmem + h * g.acc_stride, umma_desc_sw128(a + k4 * 32), umma_desc_sw128(bb + h * g.tile_n * 128 + k4 * 32), g.idesc,
                                      (kb > 0 || k4 > 0) ? 1u : 0u);
                    umma_commit(empty_bar(s));
                }
                if (ok) umma_commit(accf_bar(b));
            }
            if (!ok) atomicCAS(g.status, 0u, timeout_word(g, 2));
        }
    } else {
        const int wt = threadIdx.x - 64;
        const DwUnit du = make_dw_unit(g, wt, dw_quads, dw_br);
        const int zero_from = g.halo_cb >> 3;
        if (zero_from < 8) {
            // K-padding chunks are only ever written with zeros: cleared once
            const int nz = 8 - zero_from;
            for (int idx = wt; idx < g.stages * kTileM * nz; idx += kWorkerThreads) {
                const int sr = idx / nz, jj = zero_from + idx - sr * nz, s = sr / kTileM, row = sr - s * kTileM;
                st_shared16(a_chunk_addr(sbase + s * stage_bytes, row, jj), make_uint4(0u, 0u, 0u, 0u));
            }
            fence_proxy_async();
        }
        const uint32_t dww = sbase + g.off_dww;
        const GemmSeg &sg = g.seg[0];
        const int quarter = warp & 3, cgroup = (warp - 2) >> 2;      // accumulator lanes; which 32-column chunks
        const int row = quarter * 32 + lane;
        const RowLocal rl = row_local(g, row);
        const uint32_t plo = g.act >= 1 ? 0u : 0xff80ff80u, phi = g.act == 2 ? 0x40c040c0u : 0x7f807f80u;
        const bool wide_ok = ((reinterpret_cast<uintptr_t>(g.out) | (uintptr_t)(g.out_ctot * 2) | (uintptr_t)(g.out_coff * 2)) & 31u) == 0;
        Ring st = {0, 0u}, hr = {0, 0u};
        ok = mbar_wait_warp(dww_bar, 0u, lane);
        auto stencil = [&]() {
            for (int kb = 0; kb < g.kblocks && ok; ++kb) {
                const int s = st.s, hs = hr.s;
                ok = mbar_wait2_warp(empty_bar(s), st.ph ^ 1u, hfull_bar(hs), hr.ph, lane);
                if (!ok) break;
                st.next(g.stages); hr.next(g.hstages);
                const uint32_t a_base = sbase + s * stage_bytes, halo = sbase + g.off_halo + hs * g.halo_stride;
                if (kW == 8 && g.halo_cb > 32) {
                    if (sg.stride == 1) produce_dw<1, 2>(sg, g, kb, halo, dww, du, a_base);
                    else produce_dw<2, 2>(sg, g, kb, halo, dww, du, a_base);
                } else {
                    if (sg.stride == 1) produce_dw<1, 1>(sg, g, kb, halo, dww, du, a_base);
                    else produce_dw<2, 1>(sg, g, kb, halo, dww, du, a_base);
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) { mbar_arrive(full_bar(s)); mbar_arrive(hempty_bar(hs)); }
            }
        };
        TileWalk ws, we;
        ws.init(g);
        we.init(g);
        if (ws.ti < total_tiles) { stencil(); ws.next(g); }
        for (int i = 0; we.ti < total_tiles; we.next(g), ++i) {
            if (ok && ws.ti < total_tiles) { stencil(); ws.next(g); }
            const int b = i & 1, nt = we.nt, n0 = nt * cols;
            // the bias slice of this tile's channels (two buffers: a warp is at most one tile ahead of the others)
            // (a 512-column tile is its CTA's only tile and takes both buffers)
            const int bbuf = g.n_acc == 2 ? 0 : b;
            if (wt * 4 < cols)
                *reinterpret_cast<float4 *>(sm + g.off_bias + bbuf * 1024 + wt * 16) = __ldg(reinterpret_cast<const float4 *>(g.bias + n0) + wt);
            const uint32_t sbias = sbase + g.off_bias + bbuf * 1024;
            const RowPos rq = map_row(g, we, rl, row);
            const size_t pix = ((size_t)rq.n * g.P + rq.p) * g.Q + rq.q;
            // the workers share a named barrier, so they agree on giving up before any of them can miss it
            if (ok) ok = mbar_wait_warp(accf_bar(b), (i >> 1) & 1, lane);
            if (!ok && lane == 0) *fail_flag = 1;
            asm volatile("bar.sync 1, %0;" ::"r"(kWorkerThreads) : "memory");
            if (*fail_flag) { ok = false; break; }
            tc_fence_after();
            const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * g.acc_stride;
            const int nc32 = (cols + 31) >> 5;
            if (g.epi == GE_GAP) {
                // ---- global average of whole images (a CTA's only tile: the A|B ring is free and holds the slabs) ----
                // Per pass the kW / 4 warps of a quarter take kW / 4 chunks of 32 columns: every thread parks its row's
                // activated fp32 values in its chunk's slab [128 rows][33]; then (slab, image, column, part) items sum
                // the rows r = part, part + parts, ... in ascending order, and the parts are added in ascending order.
                constexpr int kSlabs = kW / 4;
                float *slab = reinterpret_cast<float *>(sm) + cgroup * (kTileM * 33);
                float *parts_mem = reinterpret_cast<float *>(sm) + kSlabs * (kTileM * 33);
                const float lo1 = act_lo(g.act), hi1 = act_hi(g.act);
                const int per = kSlabs * g.gap_imgs * 32;                       // (slab, image, column) triples
                const int parts = per * 4 <= kWorkerThreads ? 4 : (per * 2 <= kWorkerThreads ? 2 : 1);
                for (int c0 = 0; c0 < nc32; c0 += kSlabs) {
                    const int c32 = c0 + cgroup;
                    if (c32 < nc32) {
                        float v[32];
                        const bool whole = c32 * 32 + 32 <= cols;
                        if (whole) tmem_ld32(t_lane + c32 * 32, v);
                        else { tmem_ld16(t_lane + c32 * 32, v); for (int e = 16; e < 32; ++e) v[e] = 0.0f; }
#pragma unroll
                        for (int q4 = 0; q4 < 32; q4 += 4) {
                            float4 bz = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (c32 * 32 + q4 < cols) bz = ld_shared_f4(sbias + (uint32_t)(c32 * 32 + q4) * 4u);
                            slab[row * 33 + q4] = rq.valid ? fminf(fmaxf(v[q4] + bz.x, lo1), hi1) : 0.0f;
                            slab[row * 33 + q4 + 1] = rq.valid ? fminf(fmaxf(v[q4 + 1] + bz.y, lo1), hi1) : 0.0f;
                            slab[row * 33 + q4 + 2] = rq.valid ? fminf(fmaxf(v[q4 + 2] + bz.z, lo1), hi1) : 0.0f;
                            slab[row * 33 + q4 + 3] = rq.valid ? fminf(fmaxf(v[q4 + 3] + bz.w, lo1), hi1) : 0.0f;
                        }
                    }
                    if (c0 + kSlabs >= nc32) {
                        // this warp's last read of the accumulator
                        tc_fence_before();
                        warp_arrive(acce_bar(b), lane);
                    }
                    asm volatile("bar.sync 1, %0;" ::"r"(kWorkerThreads) : "memory");
                    for (int item = wt; item < per * parts; item += kWorkerThreads) {
                        const int c = item & 31, rest = item >> 5;
                        const int pa = rest % parts, tri = rest / parts, sl = tri % kSlabs, img = tri / kSlabs;
                        const float *src = reinterpret_cast<float *>(sm) + sl * (kTileM * 33);
                        float acc = 0.0f;
                        for (int r = pa; r < g.gap_area; r += parts) acc += src[(img * g.gap_area + r) * 33 + c];
                        parts_mem[item] = acc;
                    }
                    asm volatile("bar.sync 1, %0;" ::"r"(kWorkerThreads) : "memory");
                    for (int item = wt; item < per; item += kWorkerThreads) {
                        const int c = item & 31, tri = item >> 5, sl = tri % kSlabs, img = tri / kSlabs;
                        const int n = we.mt * g.gap_imgs + img, nc = n0 + (c0 + sl) * 32 + c;
                        if (c0 + sl >= nc32 || n >= g.batch || nc >= g.N) continue;
                        float acc = 0.0f;
                        for (int pa = 0; pa < parts; ++pa) acc += parts_mem[((tri * parts + pa) << 5) + c];
                        acc /= (float)g.gap_rpi;
                        const size_t oi = (size_t)n * g.out_ctot + g.out_coff + nc;
                        if (g.out_f32) reinterpret_cast<float *>(g.out)[oi] = acc;
                        else reinterpret_cast<__nv_bfloat16 *>(g.out)[oi] = __float2bfloat16_rn(acc);
                    }
                    // (the next pass's slab writes follow this pass's reads of parts_mem only; the slabs were last read
                    // before the barrier above)
                }
                continue;
            }
            for (int c32 = cgroup; c32 < nc32; c32 += kW / 4) {
                float v[32];
                const bool whole = c32 * 32 + 32 <= cols;
                if (whole) tmem_ld32(t_lane + c32 * 32, v);
                else tmem_ld16(t_lane + c32 * 32, v);
                if (c32 + kW / 4 >= nc32) {
                    // this warp's last read of the accumulator
                    tc_fence_before();
                    warp_arrive(acce_bar(b), lane);
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (h == 1 && !whole) break;
                    const int cl = c32 * 32 + h * 16, nc = n0 + cl;
                    uint32_t pk[8];
#pragma unroll
                    for (int q4 = 0; q4 < 16; q4 += 4) {
                        const float4 bz = ld_shared_f4(sbias + (uint32_t)(cl + q4) * 4u);
                        const float2 t0 = __fadd2_rn(make_float2(v[h * 16 + q4], v[h * 16 + q4 + 1]), make_float2(bz.x, bz.y));
                        const float2 t1 = __fadd2_rn(make_float2(v[h * 16 + q4 + 2], v[h * 16 + q4 + 3]), make_float2(bz.z, bz.w));
                        pk[q4 / 2] = clamp_bf16x2(pack2(t0.x, t0.y), plo, phi);
                        pk[q4 / 2 + 1] = clamp_bf16x2(pack2(t1.x, t1.y), plo, phi);
                    }
                    if (!rq.valid) continue;
                    __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(g.out) + pix * g.out_ctot + g.out_coff + nc;
                    if (nc + 16 <= g.N && wide_ok) {
                        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(o), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]),
                                     "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]) : "memory");
                    } else {
                        if (nc + 8 <= g.N) *reinterpret_cast<uint4 *>(o) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        if (nc + 16 <= g.N) *reinterpret_cast<uint4 *>(o + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                    }
                }
            }
            if (cgroup >= nc32) warp_arrive(acce_bar(b), lane);       // a warp without a chunk in so narrow a tile
        }
        if (!ok && lane == 0) atomicCAS(g.status, 0u, timeout_word(g, 3));
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols) : "memory");
    }
}

}  // namespace xk
