// CUDA runtime of the library: uploads the packed parameters into the caller's workspace,
// encodes the TMA descriptors, and enqueues one kernel per launch record on the caller's stream.
// Allocates no device memory.  (Section 3 of the Xenos paper: the runtime executes the optimised
// model on the parallel units on top of the operator library.)
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include "chain2_tc.cuh"
#include "dwpw_tc.cuh"
#include "gemm_tc.cuh"
#include "graph.hpp"
#include "kernels_bf16.cuh"
#include "kernels_f32.cuh"

namespace xenos {

struct Runtime {
    int device = -1;
    int sm_count = 0;
    std::vector<CUtensorMap> tmaps;     // one per launch record (used by gemm launches only)
    std::vector<CUtensorMap> hmaps;     // halo maps of linked depthwise stages / activation operand maps
    std::vector<CUtensorMap> tmaps2;    // second weight matrix of two linked convolutions
    PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
};

static xenos_status_t cuda_fail(const Graph &g, const char *what, cudaError_t e) {
    return fail(g, XENOS_E_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

static uint32_t make_idesc(int tile_n) {
    // kind::f16 instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128
    uint32_t d = 0;
    d |= 1u << 4;                       // D format f32
    d |= 1u << 7;                       // A format bf16
    d |= 1u << 10;                      // B format bf16
    d |= (uint32_t)(tile_n >> 3) << 17; // N / 8
    d |= (uint32_t)(128 >> 4) << 24;    // M / 16
    return d;
}

// 4-D map (C, W, H, N) over the NHWC bf16 input of a linked depthwise stage; box = one halo tile.
// Out-of-range coordinates read zeros, which is the convolution's zero padding.
// `images` is the extent of the outermost dimension: boxes that reach past it (the last image group of
// an odd batch) read zeros there and never touch memory behind the buffer.
static xenos_status_t encode_halo_map(const Graph &g, Runtime *rt, const Launch &L, void *base, int images, CUtensorMap *out) {
    const ASeg &a = L.seg[0];
    cuuint64_t dims[4] = {(cuuint64_t)a.C, (cuuint64_t)a.W, (cuuint64_t)a.H, (cuuint64_t)images};
    cuuint64_t strides[3] = {(cuuint64_t)a.C * 2, (cuuint64_t)a.W * a.C * 2, (cuuint64_t)a.H * a.W * a.C * 2};
    cuuint32_t box[4] = {(cuuint32_t)L.halo_cb, (cuuint32_t)L.halo_w, (cuuint32_t)L.halo_h, (cuuint32_t)L.ni};
    cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    if (((uintptr_t)base & 15u) || (strides[0] & 15u) || (box[0] * 2u) % 16u || box[1] > 256u || box[2] > 256u || box[3] > 256u)
        return fail(g, XENOS_E_CUDA, "depthwise input is not 16-byte aligned or its halo tile exceeds the TMA box limits");
    CUresult r = rt->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(g, XENOS_E_CUDA, "cuTensorMapEncodeTiled (halo) failed with code " + std::to_string((int)r));
    return XENOS_OK;
}

// Activation operand by TMA: the [pixels][C] matrix of an NHWC tensor (box = 128 rows of one 64-channel block), or the
// tensor itself as (C, W, H, N) with a box of one tile's patch; 128-byte swizzle, the layout the MMA descriptor reads.
static xenos_status_t encode_a_map(const Graph &g, Runtime *rt, const Launch &L, void *base, int images, CUtensorMap *out) {
    const ASeg &a = L.seg[0];
    CUresult r;
    if (((uintptr_t)base & 15u) || (a.C % 64)) return fail(g, XENOS_E_CUDA, "internal: activation operand is not addressable by TMA");
    if (L.a_tma == 1) {
        cuuint64_t dims[2] = {(cuuint64_t)a.C, (cuuint64_t)images * a.H * a.W};
        cuuint64_t strides[1] = {(cuuint64_t)a.C * 2};
        cuuint32_t box[2] = {64u, 128u};
        cuuint32_t estr[2] = {1u, 1u};
        r = rt->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                       CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        cuuint64_t dims[4] = {(cuuint64_t)a.C, (cuuint64_t)a.W, (cuuint64_t)a.H, (cuuint64_t)images};
        cuuint64_t strides[3] = {(cuuint64_t)a.C * 2, (cuuint64_t)a.W * a.C * 2, (cuuint64_t)a.H * a.W * a.C * 2};
        cuuint32_t box[4] = {64u, (cuuint32_t)L.patch_rw, (cuuint32_t)L.patch_rh, (cuuint32_t)L.ni};
        cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
        if (box[1] > 256u || box[2] > 256u || box[3] > 256u || box[1] * box[2] * box[3] > 128u)
            return fail(g, XENOS_E_CUDA, "internal: activation patch exceeds the TMA box limits");
        r = rt->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                       CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) return fail(g, XENOS_E_CUDA, "cuTensorMapEncodeTiled (activation operand) failed with code " + std::to_string((int)r));
    return XENOS_OK;
}

// Maps of two linked convolutions: the first one's input (C, W, H, N) with a box of the producer tile, and the two
// packed weight matrices.
static xenos_status_t encode_chain2_input(const Graph &g, Runtime *rt, const Launch &L, void *base, int images, CUtensorMap *out) {
    const ASeg &a = L.seg[0];
    if (((uintptr_t)base & 15u) || (a.C % 64)) return fail(g, XENOS_E_CUDA, "internal: activation operand is not addressable by TMA");
    cuuint64_t dims[4] = {(cuuint64_t)a.C, (cuuint64_t)a.W, (cuuint64_t)a.H, (cuuint64_t)images};
    cuuint64_t strides[3] = {(cuuint64_t)a.C * 2, (cuuint64_t)a.W * a.C * 2, (cuuint64_t)a.H * a.W * a.C * 2};
    cuuint32_t box[4] = {64u, (cuuint32_t)L.patch_rw, (cuuint32_t)L.patch_rh, 1u};
    cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    if (box[1] > 256u || box[2] > 256u || box[1] * box[2] > 128u) return fail(g, XENOS_E_CUDA, "internal: producer tile exceeds the TMA box limits");
    CUresult r = rt->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(g, XENOS_E_CUDA, "cuTensorMapEncodeTiled (linked convolutions) failed with code " + std::to_string((int)r));
    return XENOS_OK;
}

static xenos_status_t encode_weight_map(const Graph &g, Runtime *rt, void *gaddr, int kpad, int rows, int box_rows, CUtensorMap *out) {
    cuuint64_t dims[2] = {(cuuint64_t)kpad, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)kpad * 2};
    cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1u, 1u};
    if (((uintptr_t)gaddr & 15u) || (strides[0] & 15u) || box[1] > 256u || box[1] == 0u || box_rows % 16)
        return fail(g, XENOS_E_CUDA, "internal: weight tensor map fields are misaligned");
    CUresult r = rt->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, gaddr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(g, XENOS_E_CUDA, "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r));
    return XENOS_OK;
}

// 4-D map (W, H, C, N) over a small-channel NCHW image; box = one tile's input patch, all channels.
static xenos_status_t encode_stem_map(const Graph &g, Runtime *rt, const Launch &L, void *base, int images, CUtensorMap *out) {
    const ASeg &a = L.seg[0];
    const bool f32 = a.src_dtype == XENOS_DTYPE_F32;
    const cuuint64_t es = f32 ? 4 : 2;
    cuuint64_t dims[4] = {(cuuint64_t)a.W, (cuuint64_t)a.H, (cuuint64_t)a.C, (cuuint64_t)images};
    cuuint64_t strides[3] = {(cuuint64_t)a.W * es, (cuuint64_t)a.H * a.W * es, (cuuint64_t)a.C * a.H * a.W * es};
    cuuint32_t box[4] = {(cuuint32_t)L.halo_w, (cuuint32_t)L.halo_h, (cuuint32_t)a.C, 1u};
    cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    if ((strides[0] & 15u) || (strides[1] & 15u) || (strides[2] & 15u) || (box[0] * es) % 16u || box[0] > 256u || box[1] > 256u || box[2] > 256u)
        return fail(g, XENOS_E_CUDA, "internal: stem image patch violates the TMA limits");
    CUresult r = rt->encode(out, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(g, XENOS_E_CUDA, "cuTensorMapEncodeTiled (stem) failed with code " + std::to_string((int)r));
    return XENOS_OK;
}

void runtime_free(Graph &g) {
    delete static_cast<Runtime *>(g.rt);
    g.rt = nullptr;
}

xenos_status_t runtime_bind(Graph &g, void *ws, size_t bytes, void *stream_v) {
    (void)bytes;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(g, "no CUDA device (this library has no CPU fallback)", e);
    cudaDeviceProp prop;
    if ((e = cudaGetDeviceProperties(&prop, dev)) != cudaSuccess) return cuda_fail(g, "cudaGetDeviceProperties", e);
    if (prop.major != 10) return fail(g, XENOS_E_CUDA, "device is not sm_100 (B200); the kernels are built for sm_100a only");
    runtime_free(g);
    Runtime *rt = new Runtime();
    g.rt = rt;
    rt->device = dev;
    rt->sm_count = prop.multiProcessorCount;
    // parameters -> workspace, status words cleared
    if (!g.param_blob.empty())
        if ((e = cudaMemcpyAsync(ws, g.param_blob.data(), g.param_blob.size(), cudaMemcpyHostToDevice, stream)) != cudaSuccess)
            return cuda_fail(g, "parameter upload", e);
    if ((e = cudaMemsetAsync(static_cast<uint8_t *>(ws) + g.status_off, 0, 256 + g.cnt_bytes, stream)) != cudaSuccess)
        return cuda_fail(g, "status clear", e);
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return cuda_fail(g, "parameter upload sync", e);
    g.ws = ws;
    // TMA descriptors of the packed weight matrices
    bool any_gemm = false;
    int max_gemm_smem = 0, max_chain_smem = 0;
    bool any_gemm2 = false;
    for (const Launch &L : g.launches) {
        if (L.kind == LK_GEMM2) { any_gemm = any_gemm2 = true; max_gemm_smem = std::max(max_gemm_smem, L.smem_bytes); }
        if (L.kind == LK_GEMM) { any_gemm = true; max_gemm_smem = std::max(max_gemm_smem, L.smem_bytes); }
        if (L.kind == LK_F32_CONV_CONV_POOL) max_chain_smem = std::max(max_chain_smem, L.smem_bytes);
    }
    rt->tmaps.resize(g.launches.size());
    rt->hmaps.resize(g.launches.size());
    rt->tmaps2.resize(g.launches.size());
    if (any_gemm) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess)
            return fail(g, XENOS_E_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
        rt->encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
        for (size_t i = 0; i < g.launches.size(); ++i) {
            const Launch &L = g.launches[i];
            if (L.kind == LK_GEMM2) {
                xenos_status_t st = encode_weight_map(g, rt, static_cast<uint8_t *>(ws) + L.w_off, L.kblocks * 64, L.n1pad, L.n1pad, &rt->tmaps[i]);
                if (st == XENOS_OK) st = encode_weight_map(g, rt, static_cast<uint8_t *>(ws) + L.w2_off, L.kblocks2 * 64, L.npad, L.tile_n, &rt->tmaps2[i]);
                if (st == XENOS_OK && g.tensors[L.in0].input_slot < 0)
                    st = encode_chain2_input(g, rt, L, static_cast<uint8_t *>(ws) + g.place[L.in0].off, g.max_batch, &rt->hmaps[i]);
                if (st != XENOS_OK) return st;
                continue;
            }
            if (L.kind != LK_GEMM) continue;
            cuuint64_t dims[2] = {(cuuint64_t)L.kpad, (cuuint64_t)L.npad};
            cuuint64_t strides[1] = {(cuuint64_t)L.kpad * 2};
            cuuint32_t box[2] = {64u, (cuuint32_t)L.tile_n};
            cuuint32_t estr[2] = {1u, 1u};
            void *gaddr = static_cast<uint8_t *>(ws) + L.w_off;
            // host-side validation of every field the encoder or the copy engine would reject
            if (((uintptr_t)gaddr & 15u) || (strides[0] & 15u) || box[1] > 256u || box[1] == 0u || L.tile_n % 16)
                return fail(g, XENOS_E_CUDA, "internal: weight tensor map fields are misaligned");
            CUresult r = rt->encode(&rt->tmaps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, gaddr, dims, strides, box, estr,
                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return fail(g, XENOS_E_CUDA, "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r));
            if (L.a_tma && g.tensors[L.seg[0].tensor].input_slot < 0) {
                xenos_status_t st = encode_a_map(g, rt, L, static_cast<uint8_t *>(ws) + g.place[L.seg[0].tensor].off, g.max_batch, &rt->hmaps[i]);
                if (st != XENOS_OK) return st;
            }
            if (L.seg[0].mode == AM_DW && g.tensors[L.seg[0].tensor].input_slot < 0) {
                xenos_status_t st = encode_halo_map(g, rt, L, static_cast<uint8_t *>(ws) + g.place[L.seg[0].tensor].off, g.max_batch, &rt->hmaps[i]);
                if (st != XENOS_OK) return st;
            }
        }
    }
    // The opt-in limit is a per-function, per-device setting shared by every graph in the process:
    // always raise it to the device maximum so that binding one graph never lowers it for another.
    const int optin = (int)prop.sharedMemPerBlockOptin;
    if (max_gemm_smem > optin || max_chain_smem > optin)
        return fail(g, XENOS_E_CUDA, "a kernel of this plan needs more shared memory than the device offers");
    if (any_gemm)
        if ((e = cudaFuncSetAttribute(xk::gemm_chain_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, optin)) != cudaSuccess ||
            (e = cudaFuncSetAttribute(xk::gemm_chain_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, optin)) != cudaSuccess)
            return cuda_fail(g, "cudaFuncSetAttribute(gemm)", e);
    if (any_gemm)
        if ((e = cudaFuncSetAttribute(xk::dwpw_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, optin)) != cudaSuccess ||
            (e = cudaFuncSetAttribute(xk::dwpw_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, optin)) != cudaSuccess)
            return cuda_fail(g, "cudaFuncSetAttribute(dwpw)", e);
    if (any_gemm)
        if ((e = cudaFuncSetAttribute(xk::fc_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024)) != cudaSuccess)
            return cuda_fail(g, "cudaFuncSetAttribute(fc)", e);
    if (any_gemm2)
        if ((e = cudaFuncSetAttribute(xk::chain2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin)) != cudaSuccess)
            return cuda_fail(g, "cudaFuncSetAttribute(chain2)", e);
    if (max_chain_smem > 0)
        if ((e = cudaFuncSetAttribute(xk::f32_conv_conv_pool_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin)) != cudaSuccess)
            return cuda_fail(g, "cudaFuncSetAttribute(f32 chain)", e);
    return XENOS_OK;
}

static int ew_grid(long long total, int block, int sms) {
    long long b = (total + block - 1) / block;
    long long cap = (long long)sms * 16;
    if (b > cap) b = cap;
    if (b < 1) b = 1;
    return (int)b;
}

xenos_status_t runtime_run(Graph &g, int batch, const void *const *in, void *const *out, void *stream_v,
                           float *ms_per_launch) {
    Runtime *rt = static_cast<Runtime *>(g.rt);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    uint8_t *ws = static_cast<uint8_t *>(g.ws);
    unsigned int *status = reinterpret_cast<unsigned int *>(ws + g.status_off);
    auto ptr = [&](int t) -> void * {
        if (t < 0) return nullptr;
        const Tensor &x = g.tensors[t];
        if (x.input_slot >= 0) return const_cast<void *>(in[x.input_slot]);
        if (x.output_slot >= 0) return out[x.output_slot];
        return ws + g.place[t].off;
    };
    const int sms = rt->sm_count;
    std::vector<cudaEvent_t> ev;
    if (ms_per_launch) {
        ev.resize(g.launches.size() + 1);
        for (auto &e : ev)
            if (cudaEventCreate(&e) != cudaSuccess) return fail(g, XENOS_E_CUDA, "cudaEventCreate failed");
        cudaEventRecord(ev[0], stream);
    }
    for (size_t li = 0; li < g.launches.size(); ++li) {
        const Launch &L = g.launches[li];
        const int N = batch;
        switch (L.kind) {
        case LK_F32_CONV: {
            long long total = (long long)N * L.K * L.P * L.Q;
            xk::f32_conv_kernel<<<ew_grid(total, 256, sms), 256, 0, stream>>>(
                (const float *)ptr(L.in0), (const float *)(ws + L.w_off), (const float *)(ws + L.b_off), (float *)ptr(L.out),
                N, L.C, L.H, L.W, L.K, L.P, L.Q, L.k, L.stride, L.pad, L.groups, L.act);
            break;
        }
        case LK_F32_POOL: {
            long long total = (long long)N * L.C * L.P * L.Q;
            xk::f32_pool_kernel<<<ew_grid(total, 256, sms), 256, 0, stream>>>(
                (const float *)ptr(L.in0), (float *)ptr(L.out), N, L.C, L.H, L.W, L.P, L.Q, L.pool_k, L.pool_stride, L.pool_pad, L.pool_kind);
            break;
        }
        case LK_F32_GAP: {
            long long warps = (long long)N * L.C;
            xk::f32_gap_kernel<<<(int)((warps * 32 + 255) / 256), 256, 0, stream>>>((const float *)ptr(L.in0), (float *)ptr(L.out), N * L.C, L.H * L.W);
            break;
        }
        case LK_F32_ADD: {
            const Tensor &t = g.tensors[L.out];
            long long total = (long long)N * (t.is_vec ? t.c : t.c * t.h * t.w);
            xk::f32_add_kernel<<<ew_grid(total, 256, sms), 256, 0, stream>>>((const float *)ptr(L.in0), (const float *)ptr(L.in1), (float *)ptr(L.out), total, L.act);
            break;
        }
        case LK_F32_CONCAT_PART: {
            long long total = (long long)N * L.C * L.H * L.W;
            xk::f32_concat_part_kernel<<<ew_grid(total, 256, sms), 256, 0, stream>>>((const float *)ptr(L.in0), (float *)ptr(L.out), N, L.C, L.H * L.W, L.out_ctot, L.out_coff);
            break;
        }
        case LK_F32_FC:
            xk::f32_fc_kernel<<<(N * L.K + 255) / 256, 256, 0, stream>>>((const float *)ptr(L.in0), (const float *)(ws + L.w_off), (const float *)(ws + L.b_off), (float *)ptr(L.out), N, L.C, L.K, L.act);
            break;
        case LK_F32_CONV_CONV_POOL: {
            xk::F32ChainParams p;
            p.x = (const float *)ptr(L.in0); p.y = (float *)ptr(L.out);
            p.w1 = (const float *)(ws + L.w_off); p.b1 = (const float *)(ws + L.b_off);
            p.w2 = (const float *)(ws + L.w2_off); p.b2 = (const float *)(ws + L.b2_off);
            p.N = N; p.C = L.C; p.H = L.H; p.W = L.W; p.Cmid = L.Cmid; p.P = L.P; p.Q = L.Q;
            p.k = L.k; p.stride = L.stride; p.pad = L.pad; p.act1 = L.act; p.K2 = L.K2; p.act2 = L.act2;
            p.pool_kind = L.pool_kind; p.pool_k = L.pool_k; p.pool_stride = L.pool_stride; p.PP = L.PP; p.PQ = L.PQ;
            p.parts_outc = L.parts_outc; p.tile_h = L.tile_h; p.tile_w = L.tile_w; p.tiles_h = L.tiles_h; p.tiles_w = L.tiles_w;
            p.halo_h = L.halo_h; p.halo_w = L.halo_w; p.status = status;
            xk::f32_conv_conv_pool_kernel<<<N * L.grid, L.block, L.smem_bytes, stream>>>(p);
            break;
        }
        case LK_STEM3X3: {
            const int grid = N * L.grid;
            if (L.seg[0].src_dtype == XENOS_DTYPE_F32)
                xk::stem3x3_kernel<float><<<grid, 256, (size_t)L.smem_bytes, stream>>>((const float *)ptr(L.in0), (const float *)(ws + L.w_off), (const float *)(ws + L.b_off),
                    (__nv_bfloat16 *)ptr(L.out), N, L.C, L.H, L.W, L.K, L.P, L.Q, L.stride, L.pad, L.act);
            else
                xk::stem3x3_kernel<__nv_bfloat16><<<grid, 256, (size_t)L.smem_bytes, stream>>>((const __nv_bfloat16 *)ptr(L.in0), (const float *)(ws + L.w_off), (const float *)(ws + L.b_off),
                    (__nv_bfloat16 *)ptr(L.out), N, L.C, L.H, L.W, L.K, L.P, L.Q, L.stride, L.pad, L.act);
            break;
        }
        case LK_DW: {
            long long total = (long long)N * L.P * L.Q * (L.C / 8);
            xk::dw3x3_kernel<<<ew_grid(total, 256, sms), 256, 0, stream>>>(
                (const __nv_bfloat16 *)ptr(L.in0), (const float *)(ws + L.w_off), (const float *)(ws + L.b_off),
                (__nv_bfloat16 *)ptr(L.out), N, L.C, L.H, L.W, L.P, L.Q, L.stride, L.pad, L.act);
            break;
        }
        case LK_POOL: {
            long long total = (long long)N * L.P * L.Q * (L.C / 8);
            xk::pool_kernel<<<ew_grid(total, 256, sms), 256, 0, stream>>>(
                (const __nv_bfloat16 *)ptr(L.in0), (__nv_bfloat16 *)ptr(L.out), N, L.C, L.H, L.W, L.P, L.Q, L.pool_k, L.pool_stride, L.pool_pad, L.pool_kind);
            break;
        }
        case LK_GAP: {
            int total = N * (L.C / 8);
            xk::gap_kernel<<<(total + 127) / 128, 128, 0, stream>>>((const __nv_bfloat16 *)ptr(L.in0), ptr(L.out), N, L.C, L.H * L.W, L.out_dtype == XENOS_DTYPE_F32);
            break;
        }
        case LK_ADD: {
            const Tensor &t = g.tensors[L.out];
            long long n8 = (long long)N * (t.is_vec ? t.c : t.c * t.h * t.w) / 8;
            xk::add_kernel<<<ew_grid(n8, 256, sms), 256, 0, stream>>>((const __nv_bfloat16 *)ptr(L.in0), (const __nv_bfloat16 *)ptr(L.in1), (__nv_bfloat16 *)ptr(L.out), n8, L.act);
            break;
        }
        case LK_CONCAT_PART: {
            long long pixels = (long long)N * L.H * L.W;
            xk::concat_part_kernel<<<ew_grid(pixels * (L.C / 8), 256, sms), 256, 0, stream>>>((const __nv_bfloat16 *)ptr(L.in0), (__nv_bfloat16 *)ptr(L.out), pixels, L.C, L.out_ctot, L.out_coff);
            break;
        }
        case LK_MULMAC: {
            const Tensor &t = g.tensors[L.out];
            long long n8 = (long long)N * (t.is_vec ? t.c : t.c * t.h * t.w) / 8;
            xk::mulmac_kernel<<<ew_grid(n8, 256, sms), 256, 0, stream>>>((const __nv_bfloat16 *)ptr(L.in0), (const __nv_bfloat16 *)ptr(L.in1),
                                                                         (const __nv_bfloat16 *)ptr(L.in2), (__nv_bfloat16 *)ptr(L.out), n8);
            break;
        }
        case LK_F32_MULMAC: {
            const Tensor &t = g.tensors[L.out];
            long long total = (long long)N * (t.is_vec ? t.c : t.c * t.h * t.w);
            xk::f32_mulmac_kernel<<<ew_grid(total, 256, sms), 256, 0, stream>>>((const float *)ptr(L.in0), (const float *)ptr(L.in1),
                                                                                (const float *)ptr(L.in2), (float *)ptr(L.out), total);
            break;
        }
        case LK_TRANSPOSE:      // NHWC: per image [H rows][C columns] -> [C][H]
            xk::transpose_kernel<__nv_bfloat16><<<dim3((L.C + 31) / 32, (L.H + 31) / 32, N), dim3(32, 8), 0, stream>>>(
                (const __nv_bfloat16 *)ptr(L.in0), (__nv_bfloat16 *)ptr(L.out), L.H, L.C);
            break;
        case LK_F32_TRANSPOSE:  // NCHW: per image [C][H] -> [H][C]
            xk::transpose_kernel<float><<<dim3((L.H + 31) / 32, (L.C + 31) / 32, N), dim3(32, 8), 0, stream>>>(
                (const float *)ptr(L.in0), (float *)ptr(L.out), L.C, L.H);
            break;
        case LK_SLICE: {
            long long pixels = (long long)N * L.H * L.W;
            xk::slice_kernel<<<ew_grid(pixels * (L.K / 8), 256, sms), 256, 0, stream>>>((const __nv_bfloat16 *)ptr(L.in0), (__nv_bfloat16 *)ptr(L.out), pixels, L.K, L.C, L.out_coff);
            break;
        }
        case LK_F32_SLICE: {
            long long total = (long long)N * L.K * L.H * L.W;
            xk::f32_slice_kernel<<<ew_grid(total, 256, sms), 256, 0, stream>>>((const float *)ptr(L.in0), (float *)ptr(L.out), N, L.K, L.H * L.W, L.C, L.out_coff);
            break;
        }
        case LK_GEMM2: {
            xk::Chain2Params p;
            std::memset(&p, 0, sizeof p);
            p.bias1 = (const float *)(ws + L.b_off); p.bias2 = (const float *)(ws + L.b2_off);
            p.skip = (const __nv_bfloat16 *)ptr(L.skip); p.skip_ctot = L.skip >= 0 ? g.tensors[L.skip].c : 0;
            p.out = (__nv_bfloat16 *)ptr(L.out); p.status = status;
            p.batch = N; p.P = L.P; p.Q = L.Q;
            p.k1 = L.k; p.pad1 = L.pad; p.cpb1 = L.C / 64; p.kblocks1 = L.kblocks;
            p.k2 = L.k2; p.cpb2 = L.n1pad / 64; p.kblocks2 = L.kblocks2;
            p.n1pad = L.n1pad; p.N2 = L.K; p.tile_n2 = L.tile_n; p.n2_tiles = L.n_tiles;
            p.rh1 = L.patch_rh; p.rw1 = L.patch_rw; p.halo = L.halo2; p.rh2 = L.rh2; p.rw2 = L.rw2;
            p.tiles_y = L.tiles_y; p.tiles_x = L.tiles_x; p.m_tiles = N * L.tiles_y * L.tiles_x;
            p.stages = L.stages; p.stage_bytes = L.stage_bytes; p.a_box_bytes = L.a_box_bytes;
            p.off_mid = L.off_mid; p.off_bar = L.off_bar;
            p.act1 = L.act; p.act2 = L.act2; p.act3 = L.act3; p.out_ctot = L.out_ctot; p.out_coff = L.out_coff;
            p.idesc1 = make_idesc(L.n1pad); p.idesc2 = make_idesc(L.tile_n);
            p.launch_id = (int)li;
            const CUtensorMap *tma = &rt->hmaps[li];
            CUtensorMap tma_now;
            if (g.tensors[L.in0].input_slot >= 0) {
                xenos_status_t st = encode_chain2_input(g, rt, L, ptr(L.in0), N, &tma_now);
                if (st != XENOS_OK) return st;
                tma = &tma_now;
            }
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)std::min(p.m_tiles, sms)); cfg.blockDim = dim3((unsigned)xk::kC2Threads);
            cfg.dynamicSmemBytes = (size_t)L.smem_bytes; cfg.stream = stream;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            at[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = at; cfg.numAttrs = 1;
            cudaError_t le = cudaLaunchKernelEx(&cfg, xk::chain2_kernel, *tma, rt->tmaps[li], rt->tmaps2[li], p);
            if (le != cudaSuccess) return cuda_fail(g, "kernel launch", le);
            break;
        }
        case LK_GEMM: {
            if (L.fc_small) {
                const int grid = std::min(sms, (L.K + 7) / 8);
                xk::fc_small_kernel<<<grid, 256, (size_t)N * L.C * 2, stream>>>(
                    (const __nv_bfloat16 *)ptr(L.seg[0].tensor), (const __nv_bfloat16 *)(ws + L.w_off), (const float *)(ws + L.b_off), ptr(L.out), N, L.C,
                    L.kpad, L.K, L.act, L.out_dtype == XENOS_DTYPE_F32, L.out_ctot, L.out_coff);
                break;
            }
            xk::GemmParams p;
            std::memset(&p, 0, sizeof p);
            for (int s = 0; s < 2; ++s) {
                const ASeg &a = L.seg[s];
                xk::GemmSeg &d = p.seg[s];
                d.mode = a.mode; d.src = ptr(a.tensor); d.C = a.C; d.H = a.H; d.W = a.W; d.k = a.k; d.stride = a.stride; d.pad = a.pad;
                d.kelems = a.kelems; d.kblocks = a.kblocks; d.src_f32 = a.src_dtype == XENOS_DTYPE_F32; d.dw_act = a.dw_act;
                d.dw_w = (const float *)(ws + a.dw_w_off); d.dw_b = (const float *)(ws + a.dw_b_off);
            }
            p.bias = (const float *)(ws + L.b_off);
            p.skip = (const __nv_bfloat16 *)ptr(L.skip);
            p.skip_ctot = L.skip >= 0 ? g.tensors[L.skip].c : 0;
            p.out = ptr(L.out); p.status = status;
            p.batch = N; p.P = L.P; p.Q = L.Q; p.rpi = L.rows_per_image;
            p.map_mode = L.map_mode; p.tile_rows = L.tile_rows;
            p.ni = L.ni; p.rh = L.patch_rh; p.rw = L.patch_rw; p.tiles_y = L.tiles_y; p.tiles_x = L.tiles_x;
            p.step_y = L.step_y; p.step_x = L.step_x; p.off_y = L.off_y; p.off_x = L.off_x;
            p.pool_k = L.pool_k; p.pool_stride = L.pool_stride; p.PP = L.PP; p.PQ = L.PQ; p.pth = L.patch_th; p.ptw = L.patch_tw;
            p.gap_imgs = L.gap_imgs; p.gap_area = L.gap_area; p.gap_rpi = L.gap_rpi;
            p.kblocks = L.kblocks; p.stages = L.stages; p.tile_n = L.tile_n; p.n_tiles = L.n_tiles * L.ksplit; p.N = L.K;
            p.ksplit = L.ksplit; p.kb_per = L.kb_per; p.split_ld = L.npad;
            p.split_stride = (long long)N * L.rows_per_image * L.npad;
            p.split_part = reinterpret_cast<float *>(ws + g.split_off);
            p.split_cnt = reinterpret_cast<unsigned int *>(ws + L.split_cnt_off);
            p.acc_stride = L.acc_stride; p.tmem_cols = L.tmem_cols;
            p.hstages = L.hstages; p.halo_bytes = L.halo_bytes; p.halo_stride = L.halo_stride;
            p.halo_h = L.halo_h; p.halo_w = L.halo_w; p.halo_cb = L.halo_cb;
            p.stem_tma = L.stem_tma; p.stem_align = L.stem_align;
            p.a_tma = L.a_tma; p.a_box_bytes = L.a_box_bytes; p.a_cpb = L.seg[0].C / 64;
            p.off_halo = L.off_halo; p.off_stg = L.off_stg; p.off_dww = L.off_dww; p.off_bias = L.off_bias; p.off_bar = L.off_bar;
            p.n_acc = L.n_acc; p.gap_parts = L.gap_parts;
            p.act = L.act; p.act2 = L.act2; p.epi = L.epi; p.out_ctot = L.out_ctot; p.out_coff = L.out_coff;
            p.out_f32 = L.out_dtype == XENOS_DTYPE_F32;
            p.idesc = make_idesc(L.tile_n);
            p.launch_id = (int)li;
            if (L.map_mode == MAP_PATCH) p.m_tiles = ((N + L.ni - 1) / L.ni) * L.tiles_y * L.tiles_x;
            else if (L.epi == EPI_GAP) p.m_tiles = L.gap_parts > 1 ? N * L.gap_parts : (N + L.imgs_per_tile - 1) / L.imgs_per_tile;
            else p.m_tiles = (int)(((long long)N * L.rows_per_image + 127) / 128);
            // the halo tensor map of a linked depthwise stage points at the stage's input; when that
            // is a caller buffer its address is only known now
            const CUtensorMap *tmh = &rt->tmaps[li];
            CUtensorMap tmh_now;
            if (L.stem_tma) {
                // the image is a caller buffer: encode its patch map now
                if (((uintptr_t)ptr(L.seg[0].tensor) & 15u) != 0) p.stem_tma = 0;      // unaligned image: direct loads
                else {
                    xenos_status_t st = encode_stem_map(g, rt, L, ptr(L.seg[0].tensor), N, &tmh_now);
                    if (st != XENOS_OK) return st;
                    tmh = &tmh_now;
                }
            }
            if (L.a_tma) {
                if (g.tensors[L.seg[0].tensor].input_slot >= 0) {
                    // the operand is a caller buffer: its map is encoded now (rows / images beyond the batch read zeros)
                    xenos_status_t st = encode_a_map(g, rt, L, ptr(L.seg[0].tensor), N, &tmh_now);
                    if (st != XENOS_OK) return st;
                    tmh = &tmh_now;
                } else {
                    tmh = &rt->hmaps[li];
                }
            }
            if (L.seg[0].mode == AM_DW) {
                const Tensor &hx = g.tensors[L.seg[0].tensor];
                if (hx.input_slot >= 0) {
                    xenos_status_t st = encode_halo_map(g, rt, L, ptr(L.seg[0].tensor), N, &tmh_now);
                    if (st != XENOS_OK) return st;
                    tmh = &tmh_now;
                } else {
                    tmh = &rt->hmaps[li];
                }
            }
            const int grid = std::min(p.m_tiles * p.n_tiles, sms);
            // Programmatic dependent launch: the kernel may be scheduled while its predecessor in the
            // stream drains, runs its set-up (barriers, tensor memory, constant staging) and then
            // waits (griddepcontrol.wait) before it touches any activation.
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3((unsigned)L.block);
            cfg.dynamicSmemBytes = (size_t)L.smem_bytes; cfg.stream = stream;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            at[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = at; cfg.numAttrs = 1;
            cudaError_t le;
            if (L.dw_workers == 16) le = cudaLaunchKernelEx(&cfg, xk::dwpw_kernel<16>, rt->tmaps[li], *tmh, p);
            else if (L.dw_workers == 8) le = cudaLaunchKernelEx(&cfg, xk::dwpw_kernel<8>, rt->tmaps[li], *tmh, p);
            else if (L.ksplit > 1 || L.gap_parts > 1) le = cudaLaunchKernelEx(&cfg, xk::gemm_chain_kernel<1>, rt->tmaps[li], *tmh, p);
            else le = cudaLaunchKernelEx(&cfg, xk::gemm_chain_kernel<0>, rt->tmaps[li], *tmh, p);
            if (le != cudaSuccess) return cuda_fail(g, "kernel launch", le);
            break;
        }
        default:
            return fail(g, XENOS_E_UNSUPPORTED, "internal: launch record without a kernel");
        }
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(g, "kernel launch", e);
        if (ms_per_launch) cudaEventRecord(ev[li + 1], stream);
    }
    if (ms_per_launch) {
        cudaError_t e = cudaStreamSynchronize(stream);
        for (size_t li = 0; li < g.launches.size(); ++li) {
            ms_per_launch[li] = 0.0f;
            if (e == cudaSuccess) cudaEventElapsedTime(&ms_per_launch[li], ev[li], ev[li + 1]);
        }
        for (auto &x : ev) cudaEventDestroy(x);
        if (e != cudaSuccess) return cuda_fail(g, "profile synchronize", e);
    }
    return XENOS_OK;
}

xenos_status_t runtime_status(Graph &g, void *stream_v) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    cudaError_t e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(g, "stream synchronize", e);
    unsigned int word = 0;
    uint8_t *ws = static_cast<uint8_t *>(g.ws);
    if ((e = cudaMemcpy(&word, ws + g.status_off, 4, cudaMemcpyDeviceToHost)) != cudaSuccess) return cuda_fail(g, "status read", e);
    if (word == 0) return XENOS_OK;
    cudaMemset(ws + g.status_off, 0, 256 + g.cnt_bytes);      // (the arrival counters of a run that gave up are stale too)
    int code = -(int)(word & 0xffu);
    if (code == XENOS_E_TIMEOUT) {
        static const char *role[] = {"a wait", "the TMA warp", "the MMA warp", "a producer warp", "a producer warp at the last tile", "an epilogue warp"};
        const unsigned r = (word >> 8) & 0xfu;
        return fail(g, code, std::string("a kernel gave up a bounded wait (") + role[r < 6 ? r : 0] + ", launch " + std::to_string((word >> 12) & 0xfffu) + ")");
    }
    return fail(g, code, "a kernel failed an index check");
}

xenos_status_t runtime_selftest_wait_expiry(Graph &g, void *stream_v) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    unsigned int *status = reinterpret_cast<unsigned int *>(static_cast<uint8_t *>(g.ws) + g.status_off);
    xk::wait_expiry_probe_kernel<<<1, 32, 0, stream>>>(status, 4);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(g, "kernel launch", e);
    return XENOS_OK;
}

// ------------------------------------------------------------------------------------------------
// Built-in scratch: a workspace that lives inside the library image, for callers that must not
// allocate device memory themselves.
// ------------------------------------------------------------------------------------------------
constexpr size_t kBuiltinScratchBytes = 16u << 20;    // 16 MiB, held by every device that loads the library
constexpr int kMaxDevices = 64;
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];
// In host code the name g_builtin_scratch is only a handle for the symbol, not a device address;
// the address is looked up once per device and cached here.
static void *g_builtin_ptr[kMaxDevices] = {};
static uint64_t g_builtin_owner[kMaxDevices] = {};    // serial of the graph whose parameters the array holds
static std::mutex g_builtin_mutex;                    // guards the two host tables above (not the device array)

size_t runtime_builtin_scratch_bytes() { return kBuiltinScratchBytes; }

void runtime_free_builtin(Graph &g) {
    std::lock_guard<std::mutex> lock(g_builtin_mutex);
    delete static_cast<Runtime *>(g.rt_builtin);
    g.rt_builtin = nullptr;
    for (int d = 0; d < kMaxDevices; ++d)
        if (g_builtin_owner[d] == g.serial) g_builtin_owner[d] = 0;
}

xenos_status_t runtime_run_builtin(Graph &g, int batch, const void *const *in, void *const *out, void *stream_v) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(g, "no CUDA device (this library has no CPU fallback)", e);
    if (dev < 0 || dev >= kMaxDevices) return fail(g, XENOS_E_CUDA, "run_builtin_scratch: device index out of range");
    std::lock_guard<std::mutex> lock(g_builtin_mutex);
    if (!g_builtin_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_builtin_scratch);
        if (e != cudaSuccess || !p) return cuda_fail(g, "cudaGetSymbolAddress(built-in scratch)", e);
        g_builtin_ptr[dev] = p;
    }
    void *scratch = g_builtin_ptr[dev];
    // run with the graph temporarily bound to the built-in scratch; the caller's own binding
    // (xenos_graph_bind) is put back afterwards
    // (put back on every way out of this function, an exception from the bind included)
    struct Restore {
        Graph &g; void *ws, *rt;
        ~Restore() { g.rt_builtin = g.rt; g.ws = ws; g.rt = rt; }
    } restore{g, g.ws, g.rt};
    g.rt = g.rt_builtin;
    g.rt_builtin = nullptr;               // g.rt owns the built-in binding until Restore hands it back
    xenos_status_t st = XENOS_OK;
    Runtime *rb = static_cast<Runtime *>(g.rt);
    if (!rb || rb->device != dev || g_builtin_owner[dev] != g.serial) {
        // the array holds nothing or another graph's data: upload parameters, clear status, encode maps
        g_builtin_owner[dev] = 0;
        st = runtime_bind(g, scratch, kBuiltinScratchBytes, stream);
        g_builtin_owner[dev] = st == XENOS_OK ? g.serial : 0;
    } else {
        g.ws = scratch;
        // the status word keeps the last call's contents: start from zero
        if ((e = cudaMemsetAsync(static_cast<uint8_t *>(scratch) + g.status_off, 0, 256 + g.cnt_bytes, stream)) != cudaSuccess)
            st = cuda_fail(g, "status clear", e);
    }
    if (st == XENOS_OK) st = runtime_run(g, batch, in, out, stream, nullptr);
    if (st == XENOS_OK) st = runtime_status(g, stream);
    return st;
}

}  // namespace xenos
