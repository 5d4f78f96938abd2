// Host-side graph IR, fused operators, chains and launch records.
//
// Pipeline (Section 4.3 of the Xenos paper gives the order): user operators -> Conv-Bn-Relu
// pre-fusion -> operator linking (Section 4.1, Table 1) -> operator split (Section 4.2) ->
// packed parameters + workspace layout -> launch records consumed by the CUDA runtime.
#pragma once

#include <cstddef>
#include <cstdint>
#include <string>
#include <utility>
#include <vector>

#include "../../include/xenos.h"

namespace xenos {

// ---- user-level records ----------------------------------------------------------------------
struct Tensor {
    int c = 0, h = 0, w = 0;      // per image; vectors have h == w == 0
    bool is_vec = false;
    int producer = -1;            // index into Graph::ops, -1 for a graph input
    std::vector<int> consumers;   // indices into Graph::ops
    int input_slot = -1;          // >= 0: graph input number
    int output_slot = -1;         // >= 0: graph output number
    int io_dtype = XENOS_DTYPE_F32, io_layout = XENOS_LAYOUT_NCHW;   // for graph inputs / outputs
};

struct Op {
    int kind = 0;
    int cout = 0, k = 0, stride = 1, pad = 0, groups = 1, act = 0;
    std::vector<int> in;
    int out = -1;
    std::vector<float> w, bias, gamma, beta, mean, var;
    float eps = 1e-5f;
    bool has_bias = false, has_bn = false;
};

// ---- fused operators (after the CBR pre-fusion) ----------------------------------------------
enum NodeKind { NK_CONV = 1, NK_DW, NK_FC, NK_MAXPOOL, NK_AVGPOOL, NK_GAP, NK_ADD, NK_CONCAT, NK_MUL, NK_MAC, NK_TRANSPOSE, NK_SLICE };

struct Node {
    int kind = 0;
    std::vector<int> in;          // tensor ids
    int out = -1;                 // tensor id (of the LAST fused user op)
    int cin = 0, cout = 0, k = 1, stride = 1, pad = 0, act = 0;
    std::vector<float> w;         // folded: conv [cout][cin][k][k], dw [c][k][k], fc [cout][cin]
    std::vector<float> b;         // folded bias [cout] (zeros when the op had none)
    std::vector<int> user_ops;    // indices of the user ops folded into this node
    int chain = -1;
    bool from_matmul = false;     // an x.matmul with a constant right operand (lowered like a pointwise conv / fc)
};

// ---- chains (after linking) -------------------------------------------------------------------
enum ChainKind {
    CK_SINGLE = 0,          // one fused operator, its own kernel (unlinked)
    CK_CONV_CONV_POOL,      // fp32: ConvX -> Conv1x1 -> ZPooling in one CUDA-core kernel
    CK_DW_PW,               // depthwise 3x3 -> pointwise [-> global avgpool]
    CK_CONV_TAIL,           // conv [+ linked shortcut conv] [-> add -> relu] [-> max pool | global avgpool]
    CK_EXPAND_CONCAT,       // {conv1x1, conv3x3} on one input -> concat [-> max pool]
    CK_MATMUL_MATMUL,       // MatmulX -> MatmulY with constant right operands: one product with the constants multiplied
    CK_CONV_CONV            // ConvX -> ConvY with the intermediate tile in shared memory: conv -> conv1x1 | conv3x3
                            // [-> add (identity shortcut)], or squeeze -> {expand1x1 ; expand3x3} -> concat
};

struct SplitRequest { int outc = 0, h = 0, w = 0, k = 1; bool user = false; };

// A-operand source of an implicit-GEMM launch (one K segment).
enum AMode { AM_NONE = 0, AM_GATHER = 1, AM_STEM = 2, AM_DW = 3 };
struct ASeg {
    int mode = AM_NONE;
    int tensor = -1;              // source tensor id
    int C = 0, H = 0, W = 0;      // source extent per image
    int k = 1, stride = 1, pad = 0;
    int kelems = 0;               // K elements this segment contributes (taps * C, before padding)
    int kblocks = 0;              // 64-wide K blocks (each segment starts block aligned)
    int src_dtype = XENOS_DTYPE_BF16;   // AM_STEM only: F32 or BF16 NCHW
    // AM_DW: depthwise parameters in the workspace (fp32 [9][C] tap-major, bias [C]) and its act
    size_t dw_w_off = 0, dw_b_off = 0;
    int dw_act = 0;
};

enum EpiMode { EPI_STORE = 0, EPI_GAP = 1, EPI_POOL = 2 };
enum MapMode { MAP_FLAT = 0, MAP_PATCH = 1 };

// Which kernel a launch record drives.
enum LaunchKind {
    LK_GEMM = 1,          // tcgen05 implicit GEMM chain kernel
    LK_DW,                // standalone depthwise 3x3 (bf16 NHWC)
    LK_POOL,              // standalone max / avg pool (bf16 NHWC)
    LK_GAP,               // standalone global average (bf16 NHWC -> vector)
    LK_ADD,               // standalone add (+ relu)
    LK_CONCAT_PART,       // copy one concat input to its channel offset
    LK_MULMAC,            // element-wise product / multiply-accumulate (bf16 NHWC)
    LK_TRANSPOSE,         // matrix transpose per image (bf16)
    LK_SLICE,             // channels [coff, coff + C) of the input (bf16 NHWC)
    LK_F32_CONV,          // fp32 NCHW direct conv (+bias, act), any k / stride / pad, dense or depthwise
    LK_F32_POOL, LK_F32_GAP, LK_F32_ADD, LK_F32_CONCAT_PART, LK_F32_FC,
    LK_F32_CONV_CONV_POOL, // fp32 linked chain
    LK_F32_MULMAC, LK_F32_TRANSPOSE, LK_F32_SLICE,
    LK_GEMM2,             // two linked convolutions, intermediate tile in shared memory (chain2_kernel)
    LK_STEM3X3            // 3x3 convolution of an NCHW image with at most 4 channels on the CUDA cores (stem3x3_kernel)
};

struct Launch {
    int kind = 0;
    int chain = -1;
    std::vector<int> nodes;       // node indices covered
    // ---- common tensor plumbing
    int in0 = -1, in1 = -1, in2 = -1;   // input tensors (in1: second operand of add / mul / mac, in2: addend of mac)
    int out = -1;                 // output tensor
    int out_coff = 0, out_ctot = 0;   // channel offset / total channels of the stored tensor
    int act = 0;
    // ---- geometry (per image)
    int C = 0, H = 0, W = 0;      // input extent
    int K = 0, P = 0, Q = 0;      // output channels / extent of the (first) conv or of the pool
    int k = 1, stride = 1, pad = 0, groups = 1;
    int pool_kind = 0, pool_k = 0, pool_stride = 0, pool_pad = 0, PP = 0, PQ = 0;   // linked / standalone pool
    size_t w_off = 0, b_off = 0;  // parameters in the workspace
    size_t w2_off = 0, b2_off = 0;
    // ---- implicit GEMM
    ASeg seg[2];
    int kblocks = 0, kpad = 0;    // total 64-wide K blocks, padded K
    int npad = 0;                 // padded output channels (rows of the packed weight matrix)
    int tile_n = 0, n_tiles = 0, m_tiles = 0;
    int map_mode = MAP_FLAT;
    int tile_rows = 128;          // valid rows of a 128-row M tile (FLAT); PATCH: rh * rw
    int rows_per_image = 0;       // P*Q
    int imgs_per_tile = 0;        // EPI_GAP: whole images per tile
    int patch_th = 0, patch_tw = 0, patch_rh = 0, patch_rw = 0, tiles_y = 0, tiles_x = 0;  // PATCH
    int epi = EPI_STORE;
    int skip = -1;                // tensor id added in the epilogue (identity shortcut)
    int out_dtype = XENOS_DTYPE_BF16;
    int stages = 0, smem_bytes = 0, tmem_cols = 0, pipe_bytes = 0;
    int ni = 1, step_y = 0, step_x = 0, off_y = 0, off_x = 0;      // PATCH tiles: images, tile pitch, origin offset
    int gap_imgs = 0, gap_area = 0, gap_rpi = 0;                                 // global-average epilogue
    int gap_parts = 1;                                                           // > 1: an image is averaged over that many 128-row tiles
    int acc_stride = 0;                                            // columns between the two accumulators
    int hstages = 0, halo_bytes = 0, halo_stride = 0, halo_cb = 0;   // depthwise halo ring (halo_h x halo_w input pixels per image)
    int stem_tma = 0, stem_align = 1;                              // stem: image patch by TMA, x alignment in elements
    int a_tma = 0, a_box_bytes = 0;                                // activation operand by TMA: 1 matrix rows, 2 shifted patch
    int fc_small = 0;                                              // 1: fully connected layer of a small batch on the CUDA cores (fc_small_kernel)
    int dw_workers = 0;                                            // > 0: depthwise -> pointwise in dwpw_kernel with that many worker warps
    int n_acc = 1;                                                 // dwpw_kernel: channel tiles of tile_n columns per CTA (2: both accumulators hold one tile)
    // ---- two linked convolutions (LK_GEMM2): producer tile rh1 x rw1 = patch_rh x patch_rw, consumer tile rh2 x rw2
    int k2 = 1, kblocks2 = 0, n1pad = 0, halo2 = 0, rh2 = 0, rw2 = 0, act3 = 0, off_mid = 0, stage_bytes = 0;
    int off_halo = 0, off_stg = 0, off_dww = 0, off_bias = 0, off_bar = 0;                    // shared-memory layout
    // reduction split: ksplit chunks of kb_per K blocks; fp32 partial sums [chunk][pixel][npad] in the workspace's
    // split scratch, two counters (chunks arrived, chunks reduced) per (row tile, channel tile)
    int ksplit = 1, kb_per = 0;
    size_t split_cnt_off = 0;
    // ---- fp32 linked chain (conv kxk -> conv1x1 -> pool)
    int Cmid = 0, K2 = 0, act2 = 0;
    int parts_outc = 1, tile_h = 0, tile_w = 0, tiles_h = 0, tiles_w = 0;   // tile of POOL outputs
    int halo_h = 0, halo_w = 0;   // stage-1 region a full tile needs (rows, cols)
    // ---- launch shape and modelled work
    int grid = 0, block = 0;
    double flops = 0, bytes = 0;
};

struct Chain {
    int kind = CK_SINGLE;
    std::vector<int> nodes;
    std::string pattern;          // Table 1 row this chain instantiates ("-" for a single operator)
    SplitRequest split;
    std::vector<int> launches;    // indices into Graph::launches
    double flops = 0, bytes_linked = 0, bytes_unlinked = 0;
};

struct TensorPlace {
    bool materialised = false;    // lives in memory between kernels
    bool external = false;        // graph input / output: caller's buffer
    size_t off = 0, bytes = 0;    // workspace placement (max_batch images)
    int first = -1, last = -1;    // launch interval it is live over
    int dtype = XENOS_DTYPE_BF16, layout = XENOS_LAYOUT_NHWC;
};

enum State { ST_BUILD = 0, ST_COMPILED = 1, ST_BOUND = 2 };

struct LinkRequest { std::vector<int> ops; };

struct Graph {
    xenos_hw_info_t hw{148, 227 * 1024, 512, 126ll * 1024 * 1024};
    std::vector<Tensor> tensors;
    std::vector<Op> ops;
    std::vector<int> inputs, outputs;     // tensor ids in declaration order
    bool link_auto = false;
    std::vector<LinkRequest> link_requests;
    std::vector<std::pair<int, SplitRequest>> split_requests;   // (tensor id, request)
    int state = ST_BUILD;
    // ---- compiled
    int precision = 0, max_batch = 0;
    std::vector<Node> nodes;
    std::vector<int> node_of_tensor;      // tensor id -> node producing it (-1)
    std::vector<Chain> chains;
    std::vector<Launch> launches;
    std::vector<TensorPlace> place;
    std::vector<uint8_t> param_blob;      // packed parameters, uploaded to workspace offset 0
    size_t act_off = 0;                   // start of the activation arena
    size_t cnt_bytes = 0;                 // arrival counters of reduction-split launches, right behind the status words
    size_t split_off = 0, split_bytes = 0;   // fp32 partial sums of reduction-split launches (shared: launches run in turn)
    size_t status_off = 0;                // 64-byte device status area
    size_t workspace_bytes = 0;
    std::string plan_json;
    // ---- bound
    void *ws = nullptr;
    void *rt = nullptr;                   // runtime-private data (tensor maps), owned by runtime.cu
    void *rt_builtin = nullptr;           // the same for the binding to the library's built-in scratch
    uint64_t serial = 0;                  // unique per graph, names the owner of the built-in scratch
    mutable std::string err;
};

// graph.cpp
xenos_status_t infer_and_append(Graph &g, const xenos_op_desc_t &d, const int *in, int n_in, int *out);
xenos_status_t compile_graph(Graph &g, int max_batch, int precision);
// passes.cpp
xenos_status_t prefuse(Graph &g);
xenos_status_t link_pass(Graph &g);
xenos_status_t split_and_lower(Graph &g);
xenos_status_t plan_workspace(Graph &g);
void emit_plan_json(Graph &g);
uint16_t f32_to_bf16_rne(float f);
// search.cpp
xenos_status_t search_splits(Graph &g, int max_batch, int precision, void *ws, size_t ws_bytes, const void *const *in,
                             void *const *out, void *stream, int max_trials, int repeats, std::string &report);
// serialize.cpp
void save_graph(const Graph &g, std::vector<uint8_t> &out);
xenos_status_t load_graph(Graph &g, const uint8_t *buf, size_t bytes, bool *compiled);
// runtime.cu
xenos_status_t runtime_bind(Graph &g, void *ws, size_t bytes, void *stream);
xenos_status_t runtime_run(Graph &g, int batch, const void *const *in, void *const *out, void *stream,
                           float *ms_per_launch = nullptr);
xenos_status_t runtime_status(Graph &g, void *stream);
xenos_status_t runtime_selftest_wait_expiry(Graph &g, void *stream);
void runtime_free(Graph &g);
xenos_status_t runtime_run_builtin(Graph &g, int batch, const void *const *in, void *const *out, void *stream);
void runtime_free_builtin(Graph &g);
size_t runtime_builtin_scratch_bytes();

xenos_status_t fail(const Graph &g, xenos_status_t code, const std::string &msg);

inline int out_dim(int in, int k, int stride, int pad) {
    int num = in + 2 * pad - k;
    return num < 0 ? 0 : num / stride + 1;
}
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace xenos
