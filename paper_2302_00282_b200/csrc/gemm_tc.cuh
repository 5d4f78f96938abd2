// Linked-chain implicit GEMM on the 5th-generation tensor cores (sm_100a), persistent form.
//
// One CTA per SM walks over the tiles of a chain (tile = 128 output pixels x tile_n <= 256 output
// channels: the operator split of Section 4.2 of the Xenos paper, output channels first, then
// rows / columns), so that tensor-memory allocation, barrier set-up and descriptor fetches are
// paid once and the stages of neighbouring tiles overlap:
//   warp 0        : TMA producer - weight tiles (128-byte swizzle) and, for linked depthwise
//                   chains, the input halo tile of the depthwise stage (4-D box, zero fill = padding)
//   warp 1        : one lane issues tcgen05.mma (bf16 x bf16 -> fp32) into one of two
//                   tensor-memory accumulators
//   warps 2..9    : produce the activation operand straight into shared memory in the layout the
//                   tensor core reads (K-major, 128-byte swizzle) - the paper's "write in the
//                   order the next operator reads" (Section 4.1)
//   warps 10..13  : epilogue of the previous tile, overlapped with the production of the next
// The activation operand of one 64-wide K block comes from one of
//   gather : a k x k / strided / padded window of an NHWC bf16 tensor (16-byte cp.async, zero fill)
//   stem   : a k x k window of a small-channel NCHW image (scalar loads, converted to bf16)
//   dw     : a depthwise 3x3 + bias + activation computed from the halo tile in shared memory
// and a second gather segment can append the K blocks of a shortcut 1x1 convolution, so the
// residual sum of a shortcut connection happens in the accumulator.
// Epilogues: bias, activation, identity-shortcut add, then a store at a channel offset (concat
// needs no kernel), a max pool over the tile's patch, or a global average.
//
// Every wait on an mbarrier is bounded; on expiry the role records XENOS_E_TIMEOUT in the status
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
constexpr int kMaxHaloStages = 4;
constexpr int kProducerThreads = 256;           // warps 2..9
constexpr int kParts = kProducerThreads / kTileM;      // gather / stem: threads per tile row
constexpr int kChunksPerThread = 8 / kParts;    // 16-byte chunks of a row's K block per thread
constexpr int kEpilogueThreads = 128;           // the last four warps
constexpr int kThreads = 64 + kProducerThreads + kEpilogueThreads;
constexpr unsigned kStatusTimeout = 0x80000000u | 9u;
constexpr unsigned kStatusBounds = 0x80000000u | 10u;
constexpr int kSpinLimit = 1 << 16;             // try_wait polls before a wait gives up (about a second)
constexpr unsigned kSuspendHintNs = 16000;       // a waiting thread sleeps in hardware up to this long per poll,
                                                // so pollers do not take issue slots from the working warps

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
    int map_mode, tile_rows;
    // PATCH tiles: ni images x rh x rw positions of the conv output, origin (ty*step_y - off_y, tx*step_x - off_x)
    int ni, rh, rw, tiles_y, tiles_x, step_y, step_x, off_y, off_x;
    int pool_k, pool_stride, PP, PQ, pth, ptw;     // max-pool epilogue: pth x ptw pool outputs per tile
    int gap_imgs, gap_area, gap_rpi;               // global-average epilogue: whole images per tile (area rows each, rpi of them real)
    int kblocks, stages, tile_n, n_tiles, m_tiles, N;
    int acc_stride, tmem_cols;                     // two accumulators, acc_stride columns apart
    int hstages, halo_bytes, halo_stride, halo_h, halo_w, halo_cb;   // halo ring (depthwise input tile / stem image patch)
    int stem_tma, stem_align;                       // stem: patch by TMA; x origin alignment in elements
    // Activation operand by TMA where a K block of it is a box of the NHWC tensor (stride 1, channels a multiple of
    // 64): 1 = the tile's 128 rows of the [pixels][C] matrix (1x1 convolution, fc), 2 = the tile's rh x rw patch
    // shifted by the tap (k x k; out-of-range coordinates read zeros, which is the padding).  The copy engine
    // writes the 128-byte-swizzled operand layout itself and the producer warps have nothing to do.
    int a_tma, a_box_bytes, a_cpb;                  // a_cpb: 64-channel blocks per tap
    int off_halo, off_stg, off_dww, off_bias, off_bar;   // shared-memory offsets from the 1024-aligned base
    int act, act2, epi, out_ctot, out_coff, out_f32, skip_ctot;
    uint32_t idesc;
    // reduction split (Section 4.2.2: the C / R / S split, which needs an additional reduction): the K blocks are cut
    // into ksplit chunks of kb_per blocks; n_tiles counts (channel tile, chunk) pairs, chunk fastest; partial sums go to
    // split_part [chunk][output pixel][split_ld] as fp32; when all chunks of a tile have arrived (split_cnt), each
    // chunk's CTA adds the chunks, in ascending order, for its share of the tile's rows
    int ksplit, kb_per, split_ld;
    long long split_stride;
    float *split_part;
    unsigned int *split_cnt;
    int launch_id;                                  // position of this launch in the plan, reported with a give-up
    int n_acc;                                      // dwpw_kernel: channel tiles per CTA (2: one 512-column tile in both accumulators)
    // global average of images with more than 128 pixels (1x1 convolution, rows by TMA): an image is cut into gap_parts
    // tiles of 128 rows; a tile leaves its column sums in split_part [image][part][split_ld], and the tile that arrives
    // last at the image's counter (split_cnt) adds the parts in ascending order and stores the mean
    int gap_parts;
};

// Status word of a wait that gave up: the code, the role that waited (1 TMA, 2 MMA, 3 producer, 4 producer helping
// with the last tile, 5 epilogue) and the launch.
__device__ __forceinline__ unsigned timeout_word(const GemmParams &g, int role) {
    return kStatusTimeout | ((unsigned)role << 8) | (((unsigned)g.launch_id & 0xfffu) << 12);
}

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
// Bounded wait for the phase with the given parity: one plain test, then at most `limit` polls that each
// sleep in hardware up to `hint_ns`.  Returns false when it gave up.
__device__ __forceinline__ bool mbar_wait_limited(uint32_t bar, uint32_t parity, int limit, uint32_t hint_ns) {
    {
        // most waits find their phase complete: a plain test is cheaper than a suspending wait
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    for (int i = 0; i < limit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(bar), "r"(parity), "r"(hint_ns) : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    return mbar_wait_limited(bar, parity, kSpinLimit, kSuspendHintNs);
}
// One lane polls, the warp follows: keeps 32x fewer pollers on the barrier word.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, int lane) {
    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    return ok != 0;
}
// Two barriers, one poller, one broadcast.
__device__ __forceinline__ bool mbar_wait2_warp(uint32_t bar_a, uint32_t par_a, uint32_t bar_b, uint32_t par_b, int lane) {
    int ok = 1;
    if (lane == 0) ok = (mbar_wait(bar_a, par_a) && mbar_wait(bar_b, par_b)) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    return ok != 0;
}
// Every lane has finished (and fenced) its own accesses; one arrival per warp.
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane) {
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
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
__device__ __forceinline__ float4 ld_shared_f4(uint32_t src) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(src));
    return v;
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
// c0 (the innermost coordinate) must be a multiple of 8 elements; the others may be negative
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *tm, int c0, int c1, int c2, int c3, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
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

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float *v) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Programmatic dependent launch: let the next kernel of the stream be scheduled early / wait until
// the previous kernel's memory is complete and visible (no-ops without the launch attribute).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// ---- row <-> pixel -----------------------------------------------------------------------------
struct RowPos { int valid, n, p, q; };

// A ring of n slots with the phase bit of its barriers.
struct Ring {
    int s;
    uint32_t ph;
    __device__ __forceinline__ void next(int n) { if (++s == n) { s = 0; ph ^= 1u; } }
};

// Tiles are dealt round-robin: CTA b takes tiles b, b + grid, ...  The walk keeps (mt, nt) and, for
// patch tiles, (image group, tile row, tile column) current with additions and carries, so that no
// role divides inside its tile loop.
struct TileWalk {
    int ti, mt, nt, grp, ty, tx;
    int d_mt, d_nt, d_grp, d_ty, d_tx;
    __device__ __forceinline__ void init(const GemmParams &g) {
        ti = (int)blockIdx.x; mt = ti / g.n_tiles; nt = ti - mt * g.n_tiles;
        d_mt = (int)gridDim.x / g.n_tiles; d_nt = (int)gridDim.x - d_mt * g.n_tiles;
        grp = ty = tx = d_grp = d_ty = d_tx = 0;
        if (g.map_mode == GM_PATCH) {
            const int per = g.tiles_y * g.tiles_x;
            grp = mt / per;
            int t = mt - grp * per;
            ty = t / g.tiles_x; tx = t - ty * g.tiles_x;
            d_grp = d_mt / per;
            t = d_mt - d_grp * per;
            d_ty = t / g.tiles_x; d_tx = t - d_ty * g.tiles_x;
        }
    }
    __device__ __forceinline__ void next(const GemmParams &g) {
        ti += (int)gridDim.x; mt += d_mt; nt += d_nt;
        int carry = 0;
        if (nt >= g.n_tiles) { nt -= g.n_tiles; ++mt; carry = 1; }
        if (g.map_mode == GM_PATCH) {
            tx += d_tx + carry;
            if (tx >= g.tiles_x) { tx -= g.tiles_x; ++ty; }
            ty += d_ty;
            if (ty >= g.tiles_y) { ty -= g.tiles_y; ++grp; }
            grp += d_grp;
        }
    }
};

// (channel tile, K chunk) of a tile: n_tiles counts pairs when the reduction is split.
struct TileK { int nt, kb0, kb1, ks; };
template <int kSplit>
__device__ __forceinline__ TileK tile_k(const GemmParams &g, int ntv) {
    TileK t;
    t.nt = ntv; t.ks = 0; t.kb0 = 0; t.kb1 = g.kblocks;
    if (kSplit && g.ksplit > 1) {
        t.nt = ntv / g.ksplit; t.ks = ntv - t.nt * g.ksplit;
        t.kb0 = t.ks * g.kb_per; t.kb1 = min(g.kblocks, t.kb0 + g.kb_per);
    }
    return t;
}

// Position of tile row r inside a patch tile: fixed for a thread over the whole kernel.
struct RowLocal { int img, dy, dx; };

__device__ __forceinline__ RowLocal row_local(const GemmParams &g, int r) {
    RowLocal l;
    l.img = 0; l.dy = 0; l.dx = 0;
    if (g.map_mode == GM_PATCH) {
        const int area = g.rh * g.rw;
        l.img = r / area;
        const int rem = r - l.img * area;
        l.dy = rem / g.rw; l.dx = rem - l.dy * g.rw;
    }
    return l;
}

__device__ __forceinline__ RowPos map_row(const GemmParams &g, const TileWalk &w, const RowLocal &l, int r) {
    RowPos o;
    o.valid = 0; o.n = 0; o.p = 0; o.q = 0;
    if (g.map_mode == GM_FLAT) {
        const unsigned m = (unsigned)w.mt * (unsigned)g.tile_rows + (unsigned)r;     // < 2^31 rows by construction
        if (r < g.tile_rows && m < (unsigned)g.batch * (unsigned)g.rpi) {
            o.n = (int)(m / (unsigned)g.rpi);
            const int rem = (int)(m - (unsigned)o.n * (unsigned)g.rpi);
            o.p = rem / g.Q; o.q = rem - o.p * g.Q;
            o.valid = 1;
        }
    } else {
        o.n = w.grp * g.ni + l.img;
        o.p = w.ty * g.step_y - g.off_y + l.dy;
        o.q = w.tx * g.step_x - g.off_x + l.dx;
        o.valid = (l.img < g.ni) && o.n < g.batch && o.p >= 0 && o.p < g.P && o.q >= 0 && o.q < g.Q;
    }
    return o;
}

// activation as a clamp: none = (-inf, +inf), ReLU = [0, +inf), ReLU6 = [0, 6]
__device__ __forceinline__ float act_lo(int act) { return act >= 1 ? 0.0f : -INFINITY; }
__device__ __forceinline__ float act_hi(int act) { return act == 2 ? 6.0f : INFINITY; }

// ---- A-operand producers ------------------------------------------------------------------------
// A stage is 128 rows x 128 bytes; 16-byte chunk j of row r sits at r*128 + ((j ^ (r & 7)) << 4),
// which is what a 128-byte-swizzle TMA load would have written and what the MMA descriptor expects.
__device__ __forceinline__ uint32_t a_chunk_addr(uint32_t a_base, int row, int j) {
    return a_base + row * 128 + ((j ^ (row & 7)) << 4);
}

struct GatherState { int tap_r, tap_s, cc; };   // (tap, channel chunk) of a thread's next 8-channel chunk

__device__ __forceinline__ void gather_advance(GatherState &st, int n, int C8, int k) {
    if (st.tap_r >= k) return;
    st.cc += n;
    while (st.cc >= C8 && st.tap_r < k) {
        st.cc -= C8;
        if (++st.tap_s == k) { st.tap_s = 0; ++st.tap_r; }
    }
}

// gather: a thread copies ONE 16-byte chunk j of FOUR tile rows (row0, row0 + 32, ...) per K block, so
// that the eight lanes that share a row read its 128 contiguous bytes: whole lines leave L2, not a
// 16-byte piece of 32 different lines per instruction.
struct GatherRow { int pb, ih0, iw0; };      // element index and coordinates of the row's window origin

__device__ __forceinline__ GatherRow gather_row(const GemmSeg &sg, const RowPos &rp) {
    GatherRow r;
    r.ih0 = rp.p * sg.stride - sg.pad; r.iw0 = rp.q * sg.stride - sg.pad;
    r.pb = (rp.n * sg.H + r.ih0) * sg.W + r.iw0;
    if (!rp.valid) r.ih0 = -(1 << 20);       // every tap of a row outside the tile is out of range
    return r;
}

__device__ __forceinline__ void produce_gather(const GemmSeg &sg, const GatherState &st, const GatherRow (&gr)[4], uint32_t a_base,
                                               int row0, int j) {
    const __nv_bfloat16 *src = reinterpret_cast<const __nv_bfloat16 *>(sg.src);
    const bool live_tap = st.tap_r < sg.k;                 // false: K padding behind the last tap
    const int tapoff = st.tap_r * sg.W + st.tap_s;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int ih = gr[i].ih0 + st.tap_r, iw = gr[i].iw0 + st.tap_s;
        const bool live = live_tap && (unsigned)ih < (unsigned)sg.H && (unsigned)iw < (unsigned)sg.W;
        const __nv_bfloat16 *ptr = src + ((size_t)(gr[i].pb + tapoff) * sg.C + st.cc * 8);
        cp_async16(a_chunk_addr(a_base, row0 + 32 * i, j), live ? (const void *)ptr : (const void *)src, live ? 16u : 0u);
    }
}

// stem (small-channel NCHW image, fp32 or bf16).  For k > 4, K is made of (channel c, tap row r) segments of
// kp = 8 elements, K index = (c * k + r) * kp + s: the taps s of one window row,
// which are adjacent in the image, so a 16-byte operand chunk is one or two short copies and not
// eight gathered elements.  Elements s >= k of a segment meet zero weights; they read real pixels.
// Preferred form: TMA brings the tile's input patch [C][ih][iwp] to shared memory (4-D box whose x
// origin is rounded down to a 16-byte boundary; out-of-range reads are zero = padding), one patch
// per tile, prefetched through the halo ring.
// thread = (row, part); it builds the chunks j = kParts*i + part so that all parts share the real elements.
// Small kernels (k <= 4) keep the K order (tap, channel) without padding inside K, K index e = (r * k + s) * C + c,
// and gather element by element through a table of patch offsets.
__device__ __forceinline__ void produce_stem_tile_elems(const GemmSeg &sg, const GemmParams &g, int kb_local, const uint8_t *patch,
                                                  const uint8_t *tab, int xrem, uint32_t a_base, int row, int part,
                                                  const RowLocal &rl, int jlimit) {
    // tab[e] = offset of K index e (tap-major, channel-minor) inside the patch, 0xFFFF for K padding;
    // chunks >= jlimit are K padding that the caller has cleared already
    const int base = rl.img == 0 ? (rl.dy * sg.stride) * g.halo_w + xrem + rl.dx * sg.stride : 0;   // rows past the tile read pixel 0; never stored
    const float *pf = reinterpret_cast<const float *>(patch) + base;
    const unsigned short *ph = reinterpret_cast<const unsigned short *>(patch) + base;
    const uint4 *t4 = reinterpret_cast<const uint4 *>(tab) + kb_local * 8;
#pragma unroll
    for (int i = 0; i < kChunksPerThread; ++i) {
        const int j = kParts * i + part;
        if (j >= jlimit) break;
        const uint4 o4 = t4[j];
        const uint32_t ow[4] = {o4.x, o4.y, o4.z, o4.w};
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t o0 = ow[q] & 0xFFFFu, o1 = ow[q] >> 16;
            if (sg.src_f32) {
                const float v0 = o0 != 0xFFFFu ? pf[o0] : 0.f, v1 = o1 != 0xFFFFu ? pf[o1] : 0.f;
                w[q] = pack2(v0, v1);
            } else {
                const uint32_t v0 = o0 != 0xFFFFu ? (uint32_t)ph[o0] : 0u, v1 = o1 != 0xFFFFu ? (uint32_t)ph[o1] : 0u;
                w[q] = v0 | (v1 << 16);
            }
        }
        st_shared16(a_chunk_addr(a_base, row, j), make_uint4(w[0], w[1], w[2], w[3]));
    }
}


__device__ __forceinline__ void produce_stem_direct_elems(const GemmSeg &sg, int kb_local, const RowPos &rp, uint32_t a_base,
                                                    int row, int part) {
    const int ih0 = rp.p * sg.stride - sg.pad, iw0 = rp.q * sg.stride - sg.pad;
    const size_t img = (size_t)rp.n * sg.C * sg.H * sg.W;
    const float *sf = reinterpret_cast<const float *>(sg.src) + img;
    const unsigned short *sh = reinterpret_cast<const unsigned short *>(sg.src) + img;
#pragma unroll 1
    for (int i = 0; i < kChunksPerThread; ++i) {
        const int j = kParts * i + part;
        int e = kb_local * kTileK + j * 8;
        int tap = e / sg.C, c = e - tap * sg.C;
        int r = tap / sg.k, s = tap - r * sg.k;
        f8 x;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            float v = 0.0f;
            if (rp.valid && r < sg.k) {
                const int ih = ih0 + r, iw = iw0 + s;
                if (ih >= 0 && ih < sg.H && iw >= 0 && iw < sg.W) {
                    const int off = (c * sg.H + ih) * sg.W + iw;
                    v = sg.src_f32 ? __ldg(sf + off) : __uint_as_float((unsigned)__ldg(sh + off) << 16);
                }
            }
            x.v[q] = v;
            if (++c == sg.C) { c = 0; if (++s == sg.k) { s = 0; ++r; } }
        }
        st_shared16(a_chunk_addr(a_base, row, j), pack8(x));
    }
}


// Larger kernels (k = 5..8): segments of 8.
__device__ __forceinline__ int stem_kp(int k) { return 8; }

// n = 4 or 8 consecutive patch elements starting at element offset off, as bf16 pairs
__device__ __forceinline__ void stem_copy(const uint8_t *patch, bool f32, uint32_t off, int n, uint32_t *out) {
    if (f32) {
        const float *pf = reinterpret_cast<const float *>(patch) + off;
        for (int q = 0; q < n / 2; ++q) out[q] = pack2(pf[2 * q], pf[2 * q + 1]);
    } else {
        // 16-bit elements: read the covering 32-bit words and shift by the odd element
        const uint32_t *pw = reinterpret_cast<const uint32_t *>(patch) + (off >> 1);
        const uint32_t sh = (off & 1u) * 16u;
        uint32_t w0 = pw[0];
        for (int q = 0; q < n / 2; ++q) {
            const uint32_t w1 = pw[q + 1];
            out[q] = __funnelshift_r(w0, w1, sh);
            w0 = w1;
        }
    }
}

__device__ __forceinline__ void produce_stem_tile(const GemmSeg &sg, const GemmParams &g, int kb_local, const uint8_t *patch,
                                                  const uint8_t *tab, int xrem, uint32_t a_base, int row, int part,
                                                  const RowLocal &rl, int jlimit) {
    // tab[segment] = offset of the segment's first element for the tile's pixel (0, 0), ~0 for K padding;
    // chunks >= jlimit are K padding that the caller has cleared already
    const uint32_t base = rl.img == 0 ? (uint32_t)((rl.dy * sg.stride) * g.halo_w + xrem + rl.dx * sg.stride) : 0u;   // rows past the tile read pixel 0; never stored
    const uint32_t *t32 = reinterpret_cast<const uint32_t *>(tab);
    const bool f32 = sg.src_f32 != 0;
#pragma unroll
    for (int i = 0; i < kChunksPerThread; ++i) {
        const int j = kParts * i + part;
        if (j >= jlimit) break;
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        const uint32_t o = t32[kb_local * 8 + j];
        if (o != 0xFFFFFFFFu) stem_copy(patch, f32, base + o, 8, w);
        st_shared16(a_chunk_addr(a_base, row, j), make_uint4(w[0], w[1], w[2], w[3]));
    }
}

// Fallback when the image's row pitch is not a multiple of 16 bytes (TMA cannot address it): every
// thread loads its row's elements straight from global memory.
__device__ __forceinline__ void produce_stem_direct(const GemmSeg &sg, int kb_local, const RowPos &rp, uint32_t a_base,
                                                    int row, int part) {
    const int ih0 = rp.p * sg.stride - sg.pad, iw0 = rp.q * sg.stride - sg.pad;
    const size_t img = (size_t)rp.n * sg.C * sg.H * sg.W;
    const float *sf = reinterpret_cast<const float *>(sg.src) + img;
    const unsigned short *sh = reinterpret_cast<const unsigned short *>(sg.src) + img;
    const int kp = stem_kp(sg.k);
#pragma unroll 1
    for (int i = 0; i < kChunksPerThread; ++i) {
        const int j = kParts * i + part;
        const int e = kb_local * kTileK + j * 8;
        int seg = e / kp, s = e - seg * kp;
        int c = seg / sg.k, r = seg - c * sg.k;
        f8 x;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            float v = 0.0f;
            if (rp.valid && c < sg.C && s < sg.k) {
                const int ih = ih0 + r, iw = iw0 + s;
                if (ih >= 0 && ih < sg.H && iw >= 0 && iw < sg.W) {
                    const int off = (c * sg.H + ih) * sg.W + iw;
                    v = sg.src_f32 ? __ldg(sf + off) : __uint_as_float((unsigned)__ldg(sh + off) << 16);
                }
            }
            x.v[q] = v;
            if (++s == kp) { s = 0; if (++r == sg.k) { r = 0; ++c; } }
        }
        st_shared16(a_chunk_addr(a_base, row, j), pack8(x));
    }
}

// depthwise 3x3 + bias + activation from the halo tile in shared memory ([image][y][x][cb channels],
// dense bf16), rounded to bf16 and stored in the consumer's operand layout.
// A thread owns a BR x 4 block of output pixels for FOUR channels: it walks the block's input window
// once with 8-byte loads (every input value is read once per block and feeds up to 3 * BR outputs)
// and keeps the 36 tap weights in registers.  A 64-channel K block has 16 channel quads, so the 256
// producer threads cover 16 blocks of 2 x 4 pixels; with 32 or fewer channels per K block they
// cover 32 blocks of 1 x 4.
struct DwUnit {
    int q;          // channel quad inside the K block
    int base;       // byte offset of the window origin in the halo tile (channel offset included)
    int row0;       // tile row of the block's top-left output pixel
    int nrows;      // live output rows of the block (the tile may end inside it)
    int live;
};

// The unit of producer thread pt: (pixel block, channel quad) of the tile's depthwise stage.
__device__ __forceinline__ DwUnit make_dw_unit(const GemmParams &g, int pt, int dw_quads, int dw_br) {
    DwUnit du;
    du.q = pt & (dw_quads - 1);
    const int blk = pt / dw_quads;               // (image, block row, block column)
    const int upr = g.rw >> 2, upi = ((g.rh + dw_br - 1) / dw_br) * upr;
    const int img = blk / upi, rem = blk - img * upi;
    const int uy = rem / upr, ux = rem - uy * upr;
    const int S = g.seg[0].stride;
    du.live = img < g.ni && du.q * 4 < g.halo_cb;
    du.base = ((img * g.halo_h + dw_br * uy * S) * g.halo_w + 4 * ux * S) * g.halo_cb * 2 + du.q * 8;
    du.row0 = img * g.rh * g.rw + dw_br * uy * g.rw + 4 * ux;
    du.nrows = min(dw_br, max(0, g.rh - dw_br * uy));
    return du;
}

__device__ __forceinline__ uint32_t clamp_bf16x2(uint32_t v, uint32_t lo, uint32_t hi) {
    __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162 *>(&v);
    x = __hmin2(__hmax2(x, *reinterpret_cast<__nv_bfloat162 *>(&lo)), *reinterpret_cast<__nv_bfloat162 *>(&hi));
    return *reinterpret_cast<uint32_t *>(&x);
}

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    __nv_bfloat162 x = __hmax2(*reinterpret_cast<__nv_bfloat162 *>(&a), *reinterpret_cast<__nv_bfloat162 *>(&b));
    return *reinterpret_cast<uint32_t *>(&x);
}

template <int S, int BR>
__device__ __forceinline__ void produce_dw(const GemmSeg &sg, const GemmParams &g, int kb_local, uint32_t halo, uint32_t dww,
                                           const DwUnit &u, uint32_t a_base) {
    if (!u.live) return;
    const int c0 = kb_local * kTileK + u.q * 4;
    const uint32_t half = (uint32_t)(u.q & 1) * 8u;      // which 8 bytes of the 16-byte chunk
    const int j = u.q >> 1;
    if (c0 >= sg.C) {
        // K padding inside the block: zeros, so that the zero weights there never meet a NaN
        for (int a = 0; a < u.nrows; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int r = u.row0 + a * g.rw + b;
                asm volatile("st.shared.v2.b32 [%0], {%1, %1};" ::"r"(a_chunk_addr(a_base, r, j) + half), "r"(0u) : "memory");
            }
        return;
    }
    // tap weights [9][C] and the bias [C] were staged in shared memory when the CTA started
    float2 w[9][2];
#pragma unroll
    for (int t = 0; t < 9; ++t) {
        const float4 wv = ld_shared_f4(dww + (uint32_t)(t * sg.C + c0) * 4u);
        w[t][0] = make_float2(wv.x, wv.y); w[t][1] = make_float2(wv.z, wv.w);
    }
    float2 acc[BR][4][2];
    {
        const float4 bv = ld_shared_f4(dww + (uint32_t)(9 * sg.C + c0) * 4u);
#pragma unroll
        for (int a = 0; a < BR; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) { acc[a][b][0] = make_float2(bv.x, bv.y); acc[a][b][1] = make_float2(bv.z, bv.w); }
    }
    const uint32_t hb = halo + u.base;
    const int cbytes = g.halo_cb * 2;
#pragma unroll
    for (int iy = 0; iy < (BR - 1) * S + 3; ++iy) {
#pragma unroll
        for (int ci = 0; ci < 3 * S + 3; ++ci) {
            uint32_t r0, r1;
            asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(hb + (uint32_t)((iy * g.halo_w + ci) * cbytes)));
            const float2 x0 = make_float2(__uint_as_float(r0 << 16), __uint_as_float(r0 & 0xffff0000u));
            const float2 x1 = make_float2(__uint_as_float(r1 << 16), __uint_as_float(r1 & 0xffff0000u));
#pragma unroll
            for (int ry = 0; ry < 3; ++ry) {
                if ((iy - ry) % S != 0 || iy - ry < 0 || (iy - ry) / S >= BR) continue;      // resolved at compile time
                const int a = (iy - ry) / S;
#pragma unroll
                for (int sx = 0; sx < 3; ++sx) {
                    if ((ci - sx) % S != 0 || ci - sx < 0 || (ci - sx) / S >= 4) continue;
                    const int b = (ci - sx) / S;
                    acc[a][b][0] = __ffma2_rn(x0, w[ry * 3 + sx][0], acc[a][b][0]);
                    acc[a][b][1] = __ffma2_rn(x1, w[ry * 3 + sx][1], acc[a][b][1]);
                }
            }
        }
    }
    // round to bf16, then clamp: the bounds 0 and 6 are bf16 values and rounding is monotonic, so
    // this equals clamping first
    const uint32_t lo = sg.dw_act >= 1 ? 0u : 0xff80ff80u;              // 0 | -inf, as bf16 pairs
    const uint32_t hi = sg.dw_act == 2 ? 0x40c040c0u : 0x7f807f80u;     // 6 | +inf
#pragma unroll
    for (int a = 0; a < BR; ++a) {
        if (a >= u.nrows) break;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int r = u.row0 + a * g.rw + b;
            const uint32_t p0 = clamp_bf16x2(pack2(acc[a][b][0].x, acc[a][b][0].y), lo, hi);
            const uint32_t p1 = clamp_bf16x2(pack2(acc[a][b][1].x, acc[a][b][1].y), lo, hi);
            asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(a_chunk_addr(a_base, r, j) + half), "r"(p0), "r"(p1) : "memory");
        }
    }
}

// The common store epilogue (bias, one activation as a clamp, bf16) for the 16-column chunks
// [ch0, ch1) of one tile row, bias read from global memory.  The producer warps run it on the last
// tile of their CTA, when they have nothing left to produce: three warps then share each quarter
// of the accumulator's lanes.
__device__ __forceinline__ void store_chunks(const GemmParams &g, uint32_t t_lane, const float *bias_tile, int n0, int ch0, int ch1,
                                             const RowPos &rq, size_t pix, uint32_t plo, uint32_t phi, bool wide_ok) {
    for (int cbase = ch0; cbase < ch1; cbase += 2) {
        float vv[32];
        const int nsub = (cbase + 1 < ch1) ? 2 : 1;
        if (nsub == 2) tmem_ld32(t_lane + cbase * 16, vv); else tmem_ld16(t_lane + cbase * 16, vv);
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
            if (sub >= nsub) break;
            const float *v = vv + 16 * sub;
            const int ch = cbase + sub, nc = n0 + ch * 16;
            uint32_t pk[8];
#pragma unroll
            for (int q4 = 0; q4 < 16; q4 += 4) {
                const float4 bz = __ldg(reinterpret_cast<const float4 *>(bias_tile + ch * 16 + q4));
                const float2 t0 = __fadd2_rn(make_float2(v[q4], v[q4 + 1]), make_float2(bz.x, bz.y));
                const float2 t1 = __fadd2_rn(make_float2(v[q4 + 2], v[q4 + 3]), make_float2(bz.z, bz.w));
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
}

// Four adjacent columns of one output pixel: bias, activation, identity-shortcut add, second activation, store.
// (nc is a multiple of 4 and channel counts are multiples of 8, so the four columns are inside the tensor or, for
// fp32 vector outputs, checked one by one.)
__device__ __forceinline__ void finish_store4(const GemmParams &g, float4 a, const float4 bz, int nc, size_t pix) {
    const float lo1 = act_lo(g.act), hi1 = act_hi(g.act), lo2 = act_lo(g.act2), hi2 = act_hi(g.act2);
    float v[4] = {a.x + bz.x, a.y + bz.y, a.z + bz.z, a.w + bz.w};
#pragma unroll
    for (int c = 0; c < 4; ++c) v[c] = fminf(fmaxf(v[c], lo1), hi1);
    if (g.skip) {
        const uint2 sk = __ldg(reinterpret_cast<const uint2 *>(g.skip + pix * g.skip_ctot + nc));
        v[0] += __uint_as_float(sk.x << 16); v[1] += __uint_as_float(sk.x & 0xffff0000u);
        v[2] += __uint_as_float(sk.y << 16); v[3] += __uint_as_float(sk.y & 0xffff0000u);
    }
    if (g.act2) {
#pragma unroll
        for (int c = 0; c < 4; ++c) v[c] = fminf(fmaxf(v[c], lo2), hi2);
    }
    if (g.out_f32) {
        float *o = reinterpret_cast<float *>(g.out) + pix * g.out_ctot + g.out_coff + nc;
#pragma unroll
        for (int c = 0; c < 4; ++c) if (nc + c < g.N) o[c] = v[c];
    } else {
        __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(g.out) + pix * g.out_ctot + g.out_coff + nc;
        *reinterpret_cast<uint2 *>(o) = make_uint2(pack2(v[0], v[1]), pack2(v[2], v[3]));
    }
}

// The general store epilogue for 16 columns of one tile row: bias, activation, identity-shortcut add, second
// activation, then fp32 or bf16 values at the row's position (channel offset included).
__device__ __forceinline__ void finish_store16(const GemmParams &g, float *v, uint32_t sbias, int ch, int nc, const RowPos &rq, size_t pix) {
    const float lo1 = act_lo(g.act), hi1 = act_hi(g.act), lo2 = act_lo(g.act2), hi2 = act_hi(g.act2);
#pragma unroll
    for (int q4 = 0; q4 < 16; q4 += 4) {
        const float4 bz = ld_shared_f4(sbias + (uint32_t)(ch * 16 + q4) * 4u);
        v[q4] = fminf(fmaxf(v[q4] + bz.x, lo1), hi1); v[q4 + 1] = fminf(fmaxf(v[q4 + 1] + bz.y, lo1), hi1);
        v[q4 + 2] = fminf(fmaxf(v[q4 + 2] + bz.z, lo1), hi1); v[q4 + 3] = fminf(fmaxf(v[q4 + 3] + bz.w, lo1), hi1);
    }
    if (!rq.valid) return;
    // shortcut connection with an identity branch: the skip tile is read once, here
    if (g.skip) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (nc + h * 8 + 8 > g.N) break;
            const f8 sv = unpack8(__ldg(reinterpret_cast<const uint4 *>(g.skip + pix * g.skip_ctot + nc + h * 8)));
#pragma unroll
            for (int c = 0; c < 8; ++c) v[h * 8 + c] += sv.v[c];
        }
    }
    if (g.act2) {
#pragma unroll
        for (int c = 0; c < 16; ++c) v[c] = fminf(fmaxf(v[c], lo2), hi2);
    }
    if (g.out_f32) {
        float *o = reinterpret_cast<float *>(g.out) + pix * g.out_ctot + g.out_coff + nc;
#pragma unroll
        for (int c = 0; c < 16; ++c) if (nc + c < g.N) o[c] = v[c];
    } else {
        __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(g.out) + pix * g.out_ctot + g.out_coff + nc;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (nc + h * 8 + 8 > g.N) break;
            f8 pv;
#pragma unroll
            for (int c = 0; c < 8; ++c) pv.v[c] = v[h * 8 + c];
            *reinterpret_cast<uint4 *>(o + h * 8) = pack8(pv);
        }
    }
}

// Self-test of the give-up path every role uses: one thread waits, for a few short polls only, on a
// barrier that nothing ever signals, records the expiry in the status word exactly as the roles of the
// chain kernel do, and returns normally.
__global__ void wait_expiry_probe_kernel(unsigned int *status, int polls) {
    __shared__ __align__(8) unsigned long long bar;
    if (threadIdx.x == 0) {
        const uint32_t b = smem_u32(&bar);
        mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait_limited(b, 0u, polls, 1000u)) atomicCAS(status, 0u, kStatusTimeout);
    }
}

// ---- the kernel --------------------------------------------------------------------------------
// kSplit = 1: the instance that also carries the reduction-split path (launches with ksplit > 1 use it; the
// common instance is compiled without that code).
template <int kSplit>
__global__ void __launch_bounds__(kThreads, 1)
gemm_chain_kernel(const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmH, const GemmParams g) {
    extern __shared__ uint8_t smem_raw[];
    // every CTA of this grid is resident (one per SM at most), so the next kernel can be scheduled
    // as soon as they have all started: it fills SMs as they drain and waits before touching data
    pdl_launch_dependents();
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t sbase = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (sbase - raw);
    const int stage_bytes = kABytes + g.tile_n * 128;
    const uint32_t bar_base = sbase + g.off_bar;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
    auto accf_bar = [&](int b) { return bar_base + 8u * (2 * kMaxStages + b); };
    auto acce_bar = [&](int b) { return bar_base + 8u * (2 * kMaxStages + 2 + b); };
    auto hfull_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + 4 + s); };
    auto hempty_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + 4 + kMaxHaloStages + s); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(sm + g.off_bar + 8 * (2 * kMaxStages + 4 + 2 * kMaxHaloStages));
    volatile int *fail_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);      // [0] give-up flag, [1] "this CTA completes the split tile"
    // Completion of the CTA's LAST tile, for the producer warps that help with its epilogue.  They take no part in
    // the earlier tiles, so the phase parity of the accumulator barriers would tell them nothing: a parity wait
    // cannot tell the wanted phase from the one two tiles before it.
    const uint32_t lastf_bar = bar_base + 8u * (2 * kMaxStages + 4 + 2 * kMaxHaloStages) + 16u;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = g.m_tiles * g.n_tiles;
    const bool dw_mode = g.seg[0].mode == GA_DW;
    // gather stages complete through cp.async arrivals (one per thread); the others through one
    // arrival per producer warp
    const bool tma_a = g.a_tma != 0;
    const bool async_gather = g.seg[0].mode == GA_GATHER;
    // depthwise: the producer threads are (pixel block, channel quad of the K block) pairs
    const int dw_quads = g.halo_cb > 32 ? 16 : 8;
    const int dw_br = g.halo_cb > 32 ? 2 : 1;       // block rows
    // On a CTA's last tile the producer warps take two thirds of the columns of a plain store epilogue.
    const bool help_last = g.epi == GE_STORE && !g.skip && !g.act2 && !g.out_f32 && g.tile_n >= 96 && g.ksplit <= 1;
    const int help_per = (((g.tile_n / 16) + 2) / 3 + 1) & ~1;      // 16-column chunks per sharing warp, even

    if (threadIdx.x == 0) {
        // arrivals on a stage's "full" barrier: the TMA lane plus the producers of that stage (every
        // thread for cp.async gathers, every warp otherwise)
        const uint32_t prod_warps = kProducerThreads / 32;
        const uint32_t full_count = tma_a ? 1u : (async_gather ? kProducerThreads : prod_warps) + 1;
        for (int s = 0; s < g.stages; ++s) { mbar_init(full_bar(s), full_count); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), kEpilogueThreads / 32); }
        for (int s = 0; s < g.hstages; ++s) { mbar_init(hfull_bar(s), 1); mbar_init(hempty_bar(s), prod_warps); }
        mbar_init(lastf_bar, 1);
        *fail_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
        if (dw_mode || g.stem_tma) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmH) : "memory");
    }
    if (warp == 0) {
        // The TMA lane needs the barriers only: warp 0 signals that they exist and goes straight to its
        // loads, while the other warps allocate tensor memory and stage constants before they wait.
        __syncwarp();
        asm volatile("bar.arrive 3, %0;" ::"r"(kThreads) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)g.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (dw_mode && threadIdx.x >= 64 && threadIdx.x < 64 + kProducerThreads) {
        // depthwise tap weights [9][C] followed by the bias [C], fp32, once per CTA
        const int C = g.seg[0].C;
        float4 *dst = reinterpret_cast<float4 *>(sm + g.off_dww);
        const float4 *w4 = reinterpret_cast<const float4 *>(g.seg[0].dw_w), *b4 = reinterpret_cast<const float4 *>(g.seg[0].dw_b);
        for (int i = threadIdx.x - 64; i < 9 * C / 4; i += kProducerThreads) dst[i] = __ldg(w4 + i);
        for (int i = threadIdx.x - 64; i < C / 4; i += kProducerThreads) dst[9 * C / 4 + i] = __ldg(b4 + i);
    }
    if (g.stem_tma && threadIdx.x >= 64 && threadIdx.x < 64 + kProducerThreads) {
        const int C = g.seg[0].C, k = g.seg[0].k;
        if (k > 4) {
            // K segment (channel, tap row) -> offset of its first element inside the image patch [C][halo_h][halo_w]
            uint32_t *tab = reinterpret_cast<uint32_t *>(sm + g.off_dww);
            const int nseg = g.kblocks * kTileK / stem_kp(k);
            for (int sgm = threadIdx.x - 64; sgm < nseg; sgm += kProducerThreads) {
                const int c = sgm / k, r = sgm - c * k;
                tab[sgm] = c < C ? (uint32_t)(c * g.halo_h * g.halo_w + r * g.halo_w) : 0xFFFFFFFFu;
            }
        } else {
            // K index -> offset inside the image patch
            unsigned short *tab = reinterpret_cast<unsigned short *>(sm + g.off_dww);
            const int kreal = C * k * k;
            for (int e = threadIdx.x - 64; e < g.kblocks * kTileK; e += kProducerThreads) {
                const int tap = e / C, c = e - tap * C, r = tap / k, s2 = tap - r * k;
                tab[e] = e < kreal ? (unsigned short)(c * g.halo_h * g.halo_w + r * g.halo_w + s2) : (unsigned short)0xFFFFu;
            }
        }
    }
    tc_fence_before();
    if (warp != 0) asm volatile("bar.sync 3, %0;" ::"r"(kThreads) : "memory");
    tc_fence_after();
    const uint32_t tmem_base = warp != 0 ? *tmem_slot : 0u;
    bool ok = true;
    // set-up touched constants only (weights, bias, tables); activations are the previous kernel's
    if (warp != 1) pdl_wait();

    if (warp == 0) {
        // ---- TMA: weight tiles, and the depthwise halo tiles ----
        if (lane == 0) {
            TileWalk w;
            w.init(g);
            Ring st = {0, 0u}, hr = {0, 0u};
            for (; w.ti < total_tiles && ok; w.next(g)) {
                // input origin of the tile's patch (depthwise halo / stem image patch)
                const int hn = w.grp * g.ni;
                const int hy = (w.ty * g.step_y - g.off_y) * g.seg[0].stride - g.seg[0].pad;
                const int hx = (w.tx * g.step_x - g.off_x) * g.seg[0].stride - g.seg[0].pad;
                if (g.stem_tma) {
                    // one image patch per tile: [C][ih][iwp], x origin rounded down to a 16-byte boundary
                    // (stem_align is a power of two)
                    ok = mbar_wait(hempty_bar(hr.s), hr.ph ^ 1u);
                    if (!ok) break;
                    mbar_arrive_expect_tx(hfull_bar(hr.s), (uint32_t)g.halo_bytes);
                    tma_load_4d(sbase + g.off_halo + hr.s * g.halo_stride, &tmH, hx & ~(g.stem_align - 1), hy, 0, hn, hfull_bar(hr.s));
                    hr.next(g.hstages);
                }
                const TileK tk = tile_k<kSplit>(g, w.nt);
                for (int kb = tk.kb0; kb < tk.kb1 && ok; ++kb) {
                    if (dw_mode) {
                        ok = mbar_wait(hempty_bar(hr.s), hr.ph ^ 1u);
                        if (!ok) break;
                        mbar_arrive_expect_tx(hfull_bar(hr.s), (uint32_t)g.halo_bytes);
                        tma_load_4d(sbase + g.off_halo + hr.s * g.halo_stride, &tmH, kb * kTileK, hx, hy, hn, hfull_bar(hr.s));
                        hr.next(g.hstages);
                    }
                    ok = mbar_wait(empty_bar(st.s), st.ph ^ 1u);
                    if (!ok) break;
                    mbar_arrive_expect_tx(full_bar(st.s), (uint32_t)g.tile_n * 128u + (tma_a ? (uint32_t)g.a_box_bytes : 0u));
                    if (g.a_tma == 1) {
                        const int arow = (kSplit && g.gap_parts > 1) ? (w.mt / g.gap_parts) * g.gap_rpi + (w.mt % g.gap_parts) * kTileM : w.mt * g.tile_rows;
                        tma_load_2d(sbase + st.s * stage_bytes, &tmH, kb * kTileK, arow, full_bar(st.s));
                    } else if (g.a_tma == 2) {
                        const int tap = kb / g.a_cpb, cb = kb - tap * g.a_cpb;
                        const int tr = tap / g.seg[0].k, ts = tap - tr * g.seg[0].k;
                        tma_load_4d(sbase + st.s * stage_bytes, &tmH, cb * kTileK, w.tx * g.step_x - g.off_x + ts - g.seg[0].pad,
                                    w.ty * g.step_y - g.off_y + tr - g.seg[0].pad, hn, full_bar(st.s));
                    }
                    tma_load_2d(sbase + st.s * stage_bytes + kABytes, &tmB, kb * kTileK, tk.nt * g.tile_n, full_bar(st.s));
                    st.next(g.stages);
                }
            }
            if (!ok) atomicCAS(g.status, 0u, timeout_word(g, 1));
        }
    } else if (warp == 1) {
        // ---- MMA issue ----
        if (lane == 0) {
            int i = 0;
            Ring st = {0, 0u};
            for (int ti = blockIdx.x; ti < total_tiles && ok; ti += gridDim.x, ++i) {
                const int b = i & 1;
                ok = mbar_wait(acce_bar(b), ((i >> 1) & 1) ^ 1u);      // the epilogue has drained this accumulator
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + b * g.acc_stride;
                const TileK tk = tile_k<kSplit>(g, kSplit ? ti % g.n_tiles : 0);
                for (int kb = tk.kb0; kb < tk.kb1 && ok; ++kb) {
                    const int s = st.s;
                    ok = mbar_wait(full_bar(s), st.ph);
                    if (!ok) break;
                    st.next(g.stages);
                    // the activation tile was written through the generic proxy (cp.async / st.shared)
                    // and is read by the tensor core through the async proxy
                    fence_proxy_async();
                    tc_fence_after();
                    const uint32_t a = sbase + s * stage_bytes, bb = a + kABytes;
#pragma unroll
                    for (int k4 = 0; k4 < kTileK / 16; ++k4)
                        umma_bf16(d_tmem, umma_desc_sw128(a + k4 * 32), umma_desc_sw128(bb + k4 * 32), g.idesc,
                                  (kb > tk.kb0 || k4 > 0) ? 1u : 0u);
                    umma_commit(empty_bar(s));
                }
                if (ok) {
                    umma_commit(accf_bar(b));
                    if (ti + (int)gridDim.x >= total_tiles) umma_commit(lastf_bar);
                }
            }
            if (!ok) atomicCAS(g.status, 0u, timeout_word(g, 2));
        }
    } else if (warp < 2 + kProducerThreads / 32) {
        // ---- activation operand ----
        const int pt = threadIdx.x - 64;                 // 0..255
        const int grow = pt & 127, gpart = pt >> 7;      // gather / stem mapping
        DwUnit du;
        du.q = 0; du.base = 0; du.row0 = 0; du.nrows = 0; du.live = 0;
        int zero_from = 8;                               // chunks >= zero_from of every row are K padding
        if (dw_mode) {
            zero_from = g.halo_cb >> 3;
            du = make_dw_unit(g, pt, dw_quads, dw_br);
        }
        // K-padding chunks of a depthwise stage are only ever written with zeros: when no other
        // producer shares the ring they are cleared once, here, instead of with every K block
        const bool zero_once = dw_mode && g.seg[1].mode == GA_NONE;
        if (zero_once && zero_from < 8) {
            const int nz = 8 - zero_from;
            for (int idx = pt; idx < g.stages * kTileM * nz; idx += kProducerThreads) {
                const int sr = idx / nz, jj = zero_from + idx - sr * nz, s = sr / kTileM, row = sr - s * kTileM;
                st_shared16(a_chunk_addr(sbase + s * stage_bytes, row, jj), make_uint4(0u, 0u, 0u, 0u));
            }
            fence_proxy_async();      // ordered before every later arrival of this thread
        }
        const RowLocal rl = row_local(g, grow);
        TileWalk w;
        w.init(g);
        Ring st = {0, 0u}, hr = {0, 0u};
        if (g.stem_tma) {
            // ---- stem: one image patch per tile, its K blocks gathered from the patch ----
            const GemmSeg &sg = g.seg[0];
            // with a single K block its padding chunks never change: cleared once, then skipped
            int jlimit = 8;
            if (g.kblocks == 1) {
                jlimit = (sg.C * sg.k * (sg.k > 4 ? stem_kp(sg.k) : sg.k) + 7) >> 3;
                const int nz = 8 - jlimit;
                for (int idx = pt; idx < g.stages * kTileM * nz; idx += kProducerThreads) {
                    const int sr = idx / nz, jj = jlimit + idx - sr * nz, s = sr / kTileM, row = sr - s * kTileM;
                    st_shared16(a_chunk_addr(sbase + s * stage_bytes, row, jj), make_uint4(0u, 0u, 0u, 0u));
                }
                fence_proxy_async();      // ordered before every later arrival of this thread
            }
            for (; w.ti < total_tiles && ok; w.next(g)) {
                const int shs = hr.s;
                const int xrem = ((w.tx * g.step_x - g.off_x) * sg.stride - sg.pad) & (g.stem_align - 1);
                ok = mbar_wait_warp(hfull_bar(shs), hr.ph, lane);
                if (!ok) break;
                hr.next(g.hstages);
                for (int kb = 0; kb < g.kblocks && ok; ++kb) {
                    const int s = st.s;
                    ok = mbar_wait_warp(empty_bar(s), st.ph ^ 1u, lane);
                    if (!ok) break;
                    st.next(g.stages);
                    if (sg.k > 4) produce_stem_tile(sg, g, kb, sm + g.off_halo + shs * g.halo_stride, sm + g.off_dww, xrem, sbase + s * stage_bytes, grow, gpart, rl, jlimit);
                    else produce_stem_tile_elems(sg, g, kb, sm + g.off_halo + shs * g.halo_stride, sm + g.off_dww, xrem, sbase + s * stage_bytes, grow, gpart, rl, jlimit);
                    fence_proxy_async();
                    warp_arrive(full_bar(s), lane);
                }
                if (ok) warp_arrive(hempty_bar(shs), lane);      // the image patch has been read
            }
        }
        if (dw_mode) {
            // ---- depthwise stage of a linked chain: every K block comes from a halo tile ----
            const uint32_t dww = sbase + g.off_dww;
            const GemmSeg &sg = g.seg[0];
            for (; w.ti < total_tiles && ok; w.next(g)) {
                const TileK tk = tile_k<kSplit>(g, w.nt);
                for (int kb = tk.kb0; kb < tk.kb1 && ok; ++kb) {
                    const int s = st.s, hs = hr.s;
                    ok = mbar_wait2_warp(empty_bar(s), st.ph ^ 1u, hfull_bar(hs), hr.ph, lane);
                    if (!ok) break;
                    st.next(g.stages); hr.next(g.hstages);
                    const uint32_t a_base = sbase + s * stage_bytes, halo = sbase + g.off_halo + hs * g.halo_stride;
                    if (dw_br == 2) {
                        if (sg.stride == 1) produce_dw<1, 2>(sg, g, kb, halo, dww, du, a_base);
                        else produce_dw<2, 2>(sg, g, kb, halo, dww, du, a_base);
                    } else {
                        if (sg.stride == 1) produce_dw<1, 1>(sg, g, kb, halo, dww, du, a_base);
                        else produce_dw<2, 1>(sg, g, kb, halo, dww, du, a_base);
                    }
                    // K padding: chunks the block's channels do not reach must be zero, not stale
                    if (!zero_once)
                        for (int idx = pt; idx < kTileM * (8 - zero_from); idx += kProducerThreads) {
                            const int row = idx / (8 - zero_from), jj = zero_from + idx - row * (8 - zero_from);
                            st_shared16(a_chunk_addr(a_base, row, jj), make_uint4(0u, 0u, 0u, 0u));
                        }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) { mbar_arrive(full_bar(s)); mbar_arrive(hempty_bar(hs)); }     // stage filled, halo tile read
                }
            }
        }
        // ---- general form: gathers (one or two K segments), direct stem loads ----
        const int grow0 = pt >> 3, gj = pt & 7;          // gather mapping: rows grow0 + 32 i, chunk gj
        RowLocal grl[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) grl[i] = row_local(g, grow0 + 32 * i);
        for (; !g.stem_tma && !dw_mode && !tma_a && w.ti < total_tiles && ok; w.next(g)) {
            RowPos rp;
            rp.valid = 0; rp.n = 0; rp.p = 0; rp.q = 0;
            const TileK tk = tile_k<kSplit>(g, w.nt);
            if (g.seg[0].mode == GA_STEM) rp = map_row(g, w, rl, grow);
            GatherRow gr0[4], gr1[4];
            GatherState gs0 = {0, 0, 0}, gs1 = {0, 0, 0};
            if (g.seg[0].mode == GA_GATHER) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const RowPos r4 = map_row(g, w, grl[i], grow0 + 32 * i);
                    gr0[i] = gather_row(g.seg[0], r4);
                    gr1[i] = gather_row(g.seg[1], r4);       // (unused without a second segment)
                }
                if (gj + 8 * tk.kb0) gather_advance(gs0, gj + 8 * tk.kb0, g.seg[0].C >> 3, g.seg[0].k);
                if (g.seg[1].mode == GA_GATHER) {
                    // (a chunk of a split reduction may begin inside the second segment)
                    const int adv = gj + 8 * max(0, tk.kb0 - g.seg[0].kblocks);
                    if (adv) gather_advance(gs1, adv, g.seg[1].C >> 3, g.seg[1].k);
                }
            }
            for (int kb = tk.kb0; kb < tk.kb1 && ok; ++kb) {
                const int s = st.s;
                const uint32_t sph = st.ph;
                st.next(g.stages);
                const bool first = kb < g.seg[0].kblocks;
                const GemmSeg &sg = first ? g.seg[0] : g.seg[1];
                const int kbl = first ? kb : kb - g.seg[0].kblocks;
                ok = mbar_wait_warp(empty_bar(s), sph ^ 1u, lane);
                if (!ok) break;
                const uint32_t a_base = sbase + s * stage_bytes;
                if (sg.mode == GA_GATHER) {
                    if (first) { produce_gather(sg, gs0, gr0, a_base, grow0, gj); gather_advance(gs0, 8, sg.C >> 3, sg.k); }
                    else { produce_gather(sg, gs1, gr1, a_base, grow0, gj); gather_advance(gs1, 8, sg.C >> 3, sg.k); }
                    // the stage's barrier is signalled when this thread's copies have landed; the
                    // thread itself moves on to the next stage at once
                    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(full_bar(s)) : "memory");
                } else {
                    if (sg.k > 4) produce_stem_direct(sg, kbl, rp, a_base, grow, gpart);
                    else produce_stem_direct_elems(sg, kbl, rp, a_base, grow, gpart);
                    fence_proxy_async();
                    warp_arrive(full_bar(s), lane);
                }
            }
        }
        if (!ok && lane == 0) atomicCAS(g.status, 0u, timeout_word(g, 3));
        cp_async_wait<0>();      // nothing of this thread is in flight when the CTA retires
        if (help_last && ok) {
            // this CTA's last tile: which one it is, which accumulator it sits in
            TileWalk wl, last;
            wl.init(g);
            last = wl;
            int cnt = 0;
            for (; wl.ti < total_tiles; wl.next(g)) { last = wl; ++cnt; }
            if (cnt > 0) {
                const int b = (cnt - 1) & 1, quarter = warp & 3, row = quarter * 32 + lane, helper = (warp - 2) >> 2;
                const RowLocal hl = row_local(g, row);
                const RowPos rq = map_row(g, last, hl, row);
                const size_t pix = ((size_t)rq.n * g.P + rq.p) * g.Q + rq.q;
                const uint32_t plo = g.act >= 1 ? 0u : 0xff80ff80u, phi = g.act == 2 ? 0x40c040c0u : 0x7f807f80u;
                const bool wide_ok = ((reinterpret_cast<uintptr_t>(g.out) | (uintptr_t)(g.out_ctot * 2) | (uintptr_t)(g.out_coff * 2)) & 31u) == 0;
                if (mbar_wait_warp(lastf_bar, 0u, lane)) {
                    tc_fence_after();
                    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * g.acc_stride;
                    const int nch = g.tile_n / 16;
                    const int ch0 = min(nch, help_per * (1 + helper)), ch1 = min(nch, help_per * (2 + helper));
                    store_chunks(g, t_lane, g.bias + last.nt * g.tile_n, last.nt * g.tile_n, ch0, ch1, rq, pix, plo, phi, wide_ok);
                    tc_fence_before();
                } else if (lane == 0) atomicCAS(g.status, 0u, timeout_word(g, 4));
            }
        }
    } else {
        // ---- epilogue: warp w reads tensor-memory lanes 32*(w%4).. ----
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int et = threadIdx.x - (64 + kProducerThreads);      // 0..127
        const uint32_t stg = sbase + g.off_stg;
        float *stgf = reinterpret_cast<float *>(sm + g.off_stg);
        const int pool_pitch = g.tile_n * 2 + 16;
        const int nchunks = g.tile_n / 16;
        const float lo1 = act_lo(g.act), hi1 = act_hi(g.act), lo2 = act_lo(g.act2), hi2 = act_hi(g.act2);
        // the common epilogue (bias, one activation, bf16 store or pool) runs on packed pairs
        const bool fast = !g.skip && !g.act2 && !g.out_f32 && g.epi != GE_GAP;
        const uint32_t plo = g.act >= 1 ? 0u : 0xff80ff80u, phi = g.act == 2 ? 0x40c040c0u : 0x7f807f80u;
        // 32-byte stores need a 32-byte aligned row start and column offset
        const bool wide_ok = ((reinterpret_cast<uintptr_t>(g.out) | (uintptr_t)(g.out_ctot * 2) | (uintptr_t)(g.out_coff * 2)) & 31u) == 0;
        const RowLocal rl = row_local(g, row);
        TileWalk w;
        w.init(g);
        int i = 0, bias_nt = -1, bias_buf = 0;
        for (; w.ti < total_tiles; w.next(g), ++i) {
            const TileK tk = tile_k<kSplit>(g, w.nt);
            const int mt = w.mt, nt = tk.nt;
            const int b = i & 1;
            // the bias slice of this channel tile goes to shared memory when the channel tile changes
            // (two buffers: a warp is at most one tile ahead of the others)
            const bool new_bias = nt != bias_nt;
            if (new_bias) {
                bias_nt = nt; bias_buf ^= 1;
                if (et * 4 < g.tile_n)
                    *reinterpret_cast<float4 *>(sm + g.off_bias + bias_buf * 1024 + et * 16) = __ldg(reinterpret_cast<const float4 *>(g.bias + nt * g.tile_n) + et);
            }
            const uint32_t sbias = sbase + g.off_bias + bias_buf * 1024;
            RowPos rq = map_row(g, w, rl, row);
            const bool gparts = kSplit && g.gap_parts > 1;
            const int gp_img = gparts ? mt / g.gap_parts : 0, gp_t = gparts ? mt - gp_img * g.gap_parts : 0;
            if (gparts) rq.valid = gp_t * kTileM + row < g.gap_rpi;      // rows of this image inside this tile
            const int n0 = nt * g.tile_n;
            const size_t pix = ((size_t)rq.n * g.P + rq.p) * g.Q + rq.q;
            // The four epilogue warps share named barriers (bias slice, pool and average staging), so they
            // agree on giving up before any of them can reach one: a warp whose wait ran out raises the
            // flag, all four meet, and all four leave together.
            if (!mbar_wait_warp(accf_bar(b), (i >> 1) & 1, lane) && lane == 0) *fail_flag = 1;
            epi_bar();
            if (*fail_flag) { ok = false; break; }
            tc_fence_after();
            const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * g.acc_stride;
            if (kSplit && g.ksplit > 1) {
                // ---- reduction split: park this chunk's fp32 partial sums
                float *part = g.split_part + (size_t)tk.ks * g.split_stride + pix * g.split_ld + n0;
                for (int cbase = 0; cbase < nchunks; cbase += 2) {
                    float vv[32];
                    const int nsub = (cbase + 1 < nchunks) ? 2 : 1;
                    if (nsub == 2) tmem_ld32(t_lane + cbase * 16, vv); else tmem_ld16(t_lane + cbase * 16, vv);
                    if (cbase + nsub >= nchunks) {
                        tc_fence_before();
                        warp_arrive(acce_bar(b), lane);
                    }
                    if (rq.valid)
#pragma unroll
                        for (int q4 = 0; q4 < 32; q4 += 4)
                            if (q4 < nsub * 16) __stcg(reinterpret_cast<float4 *>(part + cbase * 16 + q4), make_float4(vv[q4], vv[q4 + 1], vv[q4 + 2], vv[q4 + 3]));
                }
                // Every chunk's CTA then adds the partial sums of ITS share of the tile's rows, chunks in ascending order
                // (a fixed order: the result does not depend on which CTA arrives when): the reduction's traffic
                // is spread over the CTAs that made the partial sums, and every load is a coalesced 16 bytes.
                __threadfence();
                epi_bar();
                unsigned int *cnt = g.split_cnt + 2 * ((size_t)mt * (g.n_tiles / g.ksplit) + nt);      // [arrived, reduced]
                if (et == 0) {
                    atomicAdd(cnt, 1u);
                    int seen = 0;
                    // the other chunks of this tile are consecutive tiles of the walk: they run on other units now, or
                    // on units that are finishing an earlier tile (a wait never points at a later tile, so waits cannot
                    // form a cycle); bounded like every other wait
                    for (int spin = 0; spin < (1 << 22); ++spin) {
                        if (*reinterpret_cast<volatile unsigned int *>(cnt) >= (unsigned int)g.ksplit) { seen = 1; break; }
                        __nanosleep(64);
                    }
                    fail_flag[1] = seen;
                    if (!seen) *fail_flag = 1;
                }
                epi_bar();
                if (!fail_flag[1]) { ok = false; break; }
                __threadfence();
                {
                    const int rows_per = (kTileM + g.ksplit - 1) / g.ksplit;
                    const int r0 = tk.ks * rows_per, r1 = min(kTileM, r0 + rows_per);
                    const int c4n = g.tile_n >> 2;
                    for (int idx = et; idx < (r1 - r0) * c4n; idx += kEpilogueThreads) {
                        const int rr = r0 + idx / c4n, c4 = idx - (rr - r0) * c4n;
                        const RowPos rp = map_row(g, w, row_local(g, rr), rr);
                        const int nc = n0 + c4 * 4;
                        if (!rp.valid || nc >= g.N) continue;
                        const size_t px = ((size_t)rp.n * g.P + rp.p) * g.Q + rp.q;
                        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                        for (int sp = 0; sp < g.ksplit; ++sp) {
                            const float4 x4 = __ldcg(reinterpret_cast<const float4 *>(g.split_part + (size_t)sp * g.split_stride + px * g.split_ld + nc));
                            a.x += x4.x; a.y += x4.y; a.z += x4.z; a.w += x4.w;
                        }
                        finish_store4(g, a, ld_shared_f4(sbias + (uint32_t)(c4 * 16)), nc, px);
                    }
                }
                epi_bar();
                if (et == 0) {
                    __threadfence();
                    const unsigned int old = atomicAdd(cnt + 1, 1u);
                    if (old == (unsigned int)(g.ksplit - 1)) { cnt[0] = 0u; cnt[1] = 0u; }      // all have read: ready for the next run
                }
                continue;
            }
            // (on the CTA's last tile the producer warps store the columns behind help_per)
            const int nchunks_own = (help_last && w.ti + (int)gridDim.x >= total_tiles) ? min(nchunks, help_per) : nchunks;
            for (int cbase = 0; cbase < nchunks_own; cbase += 2) {
                // two 16-column chunks per tensor-memory load where the tile has them
                float vv[32];
                const int nsub = (cbase + 1 < nchunks_own) ? 2 : 1;
                if (nsub == 2) tmem_ld32(t_lane + cbase * 16, vv); else tmem_ld16(t_lane + cbase * 16, vv);
                if (cbase + nsub >= nchunks_own) {
                    // every column of this accumulator is in registers: hand it back to the MMA warp
                    tc_fence_before();
                    warp_arrive(acce_bar(b), lane);
                }
#pragma unroll
                for (int sub = 0; sub < 2; ++sub) {
                    if (sub >= nsub) break;
                    float *v = vv + 16 * sub;
                    const int ch = cbase + sub;
                    const int nc = n0 + ch * 16;
                    if (fast) {
                        // bias as packed fp32 adds, rounding to bf16 pairs, activation as a clamp on the pairs
                        // (0 and 6 are bf16 values and rounding is monotonic: same result as clamping first)
                        uint32_t pk[8];
#pragma unroll
                        for (int q4 = 0; q4 < 16; q4 += 4) {
                            const float4 bz = ld_shared_f4(sbias + (uint32_t)(ch * 16 + q4) * 4u);
                            const float2 t0 = __fadd2_rn(make_float2(v[q4], v[q4 + 1]), make_float2(bz.x, bz.y));
                            const float2 t1 = __fadd2_rn(make_float2(v[q4 + 2], v[q4 + 3]), make_float2(bz.z, bz.w));
                            pk[q4 / 2] = clamp_bf16x2(pack2(t0.x, t0.y), plo, phi);
                            pk[q4 / 2 + 1] = clamp_bf16x2(pack2(t1.x, t1.y), plo, phi);
                        }
                        if (g.epi == GE_STORE) {
                            if (!rq.valid) continue;
                            __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(g.out) + pix * g.out_ctot + g.out_coff + nc;
                            if (nc + 16 <= g.N && wide_ok) {
                                asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(o), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]),
                                             "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]) : "memory");
                            } else {
                                if (nc + 8 <= g.N) *reinterpret_cast<uint4 *>(o) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                                if (nc + 16 <= g.N) *reinterpret_cast<uint4 *>(o + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                            }
                        } else {
                            // rows outside the conv output never win a max
                            if (!rq.valid) {
#pragma unroll
                                for (int q = 0; q < 8; ++q) pk[q] = 0xff80ff80u;
                            }
                            st_shared16(stg + row * pool_pitch + ch * 32, make_uint4(pk[0], pk[1], pk[2], pk[3]));
                            st_shared16(stg + row * pool_pitch + ch * 32 + 16, make_uint4(pk[4], pk[5], pk[6], pk[7]));
                        }
                        continue;
                    }
                    if (g.epi == GE_STORE) { finish_store16(g, v, sbias, ch, nc, rq, pix); continue; }
                    // (pool and global-average tiles: bias, activation, [identity shortcut, activation], values kept)
#pragma unroll
                    for (int q4 = 0; q4 < 16; q4 += 4) {
                        const float4 bz = ld_shared_f4(sbias + (uint32_t)(ch * 16 + q4) * 4u);
                        v[q4] = fminf(fmaxf(v[q4] + bz.x, lo1), hi1); v[q4 + 1] = fminf(fmaxf(v[q4 + 1] + bz.y, lo1), hi1);
                        v[q4 + 2] = fminf(fmaxf(v[q4 + 2] + bz.z, lo1), hi1); v[q4 + 3] = fminf(fmaxf(v[q4 + 3] + bz.w, lo1), hi1);
                    }
                    if (g.skip && rq.valid) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if (nc + h * 8 + 8 > g.N) break;
                            const f8 sv = unpack8(__ldg(reinterpret_cast<const uint4 *>(g.skip + pix * g.skip_ctot + nc + h * 8)));
#pragma unroll
                            for (int c = 0; c < 8; ++c) v[h * 8 + c] += sv.v[c];
                        }
                    }
                    if (g.act2) {
#pragma unroll
                        for (int c = 0; c < 16; ++c) v[c] = fminf(fmaxf(v[c], lo2), hi2);
                    }
                    if (g.epi == GE_POOL) {
                        // rows outside the conv output never win a max
                        f8 lo, hi;
#pragma unroll
                        for (int c = 0; c < 8; ++c) { lo.v[c] = rq.valid ? v[c] : -INFINITY; hi.v[c] = rq.valid ? v[8 + c] : -INFINITY; }
                        st_shared16(stg + row * pool_pitch + ch * 32, pack8(lo));
                        st_shared16(stg + row * pool_pitch + ch * 32 + 16, pack8(hi));
                    }
                    // (global average: the activated values stay in vv for the reduction below)
                }
                if (g.epi == GE_GAP) {
                    // global average of up to 32 columns through shared memory: every thread parks its
                    // row, then (image, column, part) items sum the rows r = part, part + parts, ... in
                    // ascending order and the parts are added in ascending order: a fixed order
                    const int ncols = nsub * 16, nc0 = n0 + cbase * 16;
                    const int per = g.gap_imgs * 32;
                    const int parts = per >= 128 ? 1 : (per >= 64 ? 2 : 4);
                    float *part = stgf + kTileM * 33;
                    epi_bar();          // the previous slab's readers are done
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (c < ncols) stgf[row * 33 + c] = rq.valid ? vv[c] : 0.0f;
                    epi_bar();
                    for (int item = et; item < per * parts; item += kEpilogueThreads) {
                        const int c = item & 31, rest = item >> 5;
                        const int img = rest / parts, pa = rest - img * parts;
                        float acc = 0.0f;
                        if (c < ncols)
                            for (int r = pa; r < g.gap_area; r += parts) acc += stgf[(img * g.gap_area + r) * 33 + c];
                        if (parts > 1) { part[item] = acc; continue; }
                        const int n = mt * g.gap_imgs + img;
                        if (c >= ncols || n >= g.batch || nc0 + c >= g.N) continue;
                        acc /= (float)g.gap_rpi;
                        const size_t oi = (size_t)n * g.out_ctot + g.out_coff + nc0 + c;
                        if (g.out_f32) reinterpret_cast<float *>(g.out)[oi] = acc;
                        else reinterpret_cast<__nv_bfloat16 *>(g.out)[oi] = __float2bfloat16_rn(acc);
                    }
                    if (parts > 1) {
                        epi_bar();
                        for (int item = et; item < per; item += kEpilogueThreads) {
                            const int c = item & 31, img = item >> 5;
                            const int n = gparts ? gp_img : mt * g.gap_imgs + img;
                            if (c >= ncols || n >= g.batch || nc0 + c >= g.N) continue;
                            float acc = 0.0f;
                            for (int pa = 0; pa < parts; ++pa) acc += part[((img * parts + pa) << 5) + c];
                            if (gparts) {
                                // this tile's share of the image's column sum
                                __stcg(g.split_part + ((size_t)gp_img * g.gap_parts + gp_t) * g.split_ld + nc0 + c, acc);
                                continue;
                            }
                            acc /= (float)g.gap_rpi;
                            const size_t oi = (size_t)n * g.out_ctot + g.out_coff + nc0 + c;
                            if (g.out_f32) reinterpret_cast<float *>(g.out)[oi] = acc;
                            else reinterpret_cast<__nv_bfloat16 *>(g.out)[oi] = __float2bfloat16_rn(acc);
                        }
                    }
                }
            }
            if (gparts) {
                // the image's tiles meet at its counter; the one that arrives last adds the parts in ascending order
                __threadfence();
                epi_bar();
                unsigned int *cnt = g.split_cnt + 2 * ((size_t)gp_img * g.n_tiles + nt);
                if (et == 0) fail_flag[1] = atomicAdd(cnt, 1u) == (unsigned int)(g.gap_parts - 1) ? 1 : 0;
                epi_bar();
                if (fail_flag[1]) {
                    __threadfence();
                    for (int col = et; col < g.tile_n; col += kEpilogueThreads) {
                        const int nc = n0 + col;
                        if (nc >= g.N || gp_img >= g.batch) continue;
                        float acc = 0.0f;
                        for (int t = 0; t < g.gap_parts; ++t) acc += __ldcg(g.split_part + ((size_t)gp_img * g.gap_parts + t) * g.split_ld + nc);
                        acc /= (float)g.gap_rpi;
                        const size_t oi = (size_t)gp_img * g.out_ctot + g.out_coff + nc;
                        if (g.out_f32) reinterpret_cast<float *>(g.out)[oi] = acc;
                        else reinterpret_cast<__nv_bfloat16 *>(g.out)[oi] = __float2bfloat16_rn(acc);
                    }
                    if (et == 0) *cnt = 0u;      // ready for the next run
                }
                epi_bar();      // (fail_flag[1] is read before the next tile rewrites it)
            }
            if (g.epi == GE_POOL) {
                epi_bar();
                const int n = w.grp, ty = w.ty, tx = w.tx;      // pool tiles hold one image
                const int c8n = g.tile_n / 8;
                for (int item = et; item < g.pth * g.ptw * c8n; item += kEpilogueThreads) {
                    const int c8 = item % c8n, o = item / c8n;
                    const int oy = o / g.ptw, ox = o - oy * g.ptw;
                    const int gy = ty * g.pth + oy, gx = tx * g.ptw + ox;
                    const int col = n0 + c8 * 8;
                    if (gy >= g.PP || gx >= g.PQ || col + 8 > g.N || n >= g.batch) continue;
                    // the maximum of bf16 values is taken on the packed pairs (comparisons only: exact)
                    uint4 m = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);      // -inf
                    const uint32_t win = stg + (uint32_t)((oy * g.pool_stride) * g.rw + ox * g.pool_stride) * pool_pitch + c8 * 16;
                    for (int dy = 0; dy < g.pool_k; ++dy)
                        for (int dx = 0; dx < g.pool_k; ++dx) {
                            const uint4 xv = ld_shared16(win + (uint32_t)(dy * g.rw + dx) * pool_pitch);
                            m.x = max_bf16x2(m.x, xv.x); m.y = max_bf16x2(m.y, xv.y);
                            m.z = max_bf16x2(m.z, xv.z); m.w = max_bf16x2(m.w, xv.w);
                        }
                    __nv_bfloat16 *o2 = reinterpret_cast<__nv_bfloat16 *>(g.out) +
                                        (((size_t)n * g.PP + gy) * g.PQ + gx) * g.out_ctot + g.out_coff + col;
                    *reinterpret_cast<uint4 *>(o2) = m;
                }
                epi_bar();          // the staging tile is free for the next tile
            }
        }
        if (!ok && lane == 0) atomicCAS(g.status, 0u, timeout_word(g, 5));
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols) : "memory");
    }
}

}  // namespace xk
