// Host passes: Conv-Bn-Relu pre-fusion (Section 4.3), operator linking (Section 4.1, Table 1),
// operator split and lowering to launch records (Section 4.2, Eq. 1), parameter packing.
// Everything here is integer / host fp work and is deterministic: equal graphs give equal plans.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <set>

#include "graph.hpp"

namespace xenos {

uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return (uint16_t)(u >> 16);   // inf / nan: truncate
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static size_t blob_reserve(Graph &g, size_t bytes) {
    size_t off = align_up(g.param_blob.size(), 256);
    g.param_blob.resize(off + bytes, 0);
    return off;
}

// ------------------------------------------------------------------------------------------------
// Pre-fusion: Conv + Bn + Bias + Relu -> one CBR operator (Section 4.3).  BatchNorm is folded
// into the convolution: w' = w * gamma / sqrt(var + eps), b' = beta + (b - mean) * gamma / sqrt(var + eps).
// ------------------------------------------------------------------------------------------------
static void fold_bn(Node &n, const Op &bn, int per_out) {
    for (int k = 0; k < n.cout; ++k) {
        double s = (double)bn.gamma[k] / std::sqrt((double)bn.var[k] + (double)bn.eps);
        for (int i = 0; i < per_out; ++i) n.w[(size_t)k * per_out + i] = (float)((double)n.w[(size_t)k * per_out + i] * s);
        n.b[k] = (float)((double)bn.beta[k] + ((double)n.b[k] - (double)bn.mean[k]) * s);
    }
}

xenos_status_t prefuse(Graph &g) {
    g.nodes.clear();
    g.node_of_tensor.assign(g.tensors.size(), -1);
    auto sole_consumer_ok = [&](int t) {
        return g.tensors[t].consumers.size() == 1 && g.tensors[t].output_slot < 0;
    };
    for (int oi = 0; oi < (int)g.ops.size(); ++oi) {
        const Op &op = g.ops[oi];
        const Tensor &x = g.tensors[op.in[0]];
        int src = g.node_of_tensor[op.in[0]];
        switch (op.kind) {
        case XENOS_OP_CONV:
        case XENOS_OP_FC:
        case XENOS_OP_MATMUL: {
            Node n;
            n.kind = op.kind == XENOS_OP_FC ? NK_FC : (op.groups == 1 ? NK_CONV : NK_DW);
            if (op.kind == XENOS_OP_MATMUL) { n.kind = x.is_vec ? NK_FC : NK_CONV; n.from_matmul = true; }
            n.in = op.in; n.out = op.out;
            n.cin = x.c; n.cout = op.cout; n.k = op.k; n.stride = op.stride; n.pad = op.pad; n.act = op.act;
            n.w = op.w;
            n.b.assign(op.cout, 0.0f);
            if (op.has_bias) n.b = op.bias;
            if (op.has_bn) fold_bn(n, op, (int)(n.w.size() / op.cout));
            n.user_ops.push_back(oi);
            g.nodes.push_back(std::move(n));
            g.node_of_tensor[op.out] = (int)g.nodes.size() - 1;
            break;
        }
        case XENOS_OP_BATCHNORM: {
            if (src < 0 || !sole_consumer_ok(op.in[0]) || g.nodes[src].act != XENOS_ACT_NONE ||
                !(g.nodes[src].kind == NK_CONV || g.nodes[src].kind == NK_DW || g.nodes[src].kind == NK_FC))
                return fail(g, XENOS_E_UNSUPPORTED,
                            "BatchNorm that does not directly follow a convolution / fc (single consumer, no activation between) has no kernel");
            Node &n = g.nodes[src];
            fold_bn(n, op, (int)(n.w.size() / n.cout));
            g.node_of_tensor[n.out] = -1;
            n.out = op.out;
            n.user_ops.push_back(oi);
            g.node_of_tensor[op.out] = src;
            break;
        }
        case XENOS_OP_RELU:
        case XENOS_OP_RELU6: {
            if (src < 0 || !sole_consumer_ok(op.in[0]) || g.nodes[src].act != XENOS_ACT_NONE ||
                !(g.nodes[src].kind == NK_CONV || g.nodes[src].kind == NK_DW || g.nodes[src].kind == NK_FC ||
                  g.nodes[src].kind == NK_ADD))
                return fail(g, XENOS_E_UNSUPPORTED,
                            "activation that does not directly follow a convolution, fc or add (single consumer) has no kernel");
            Node &n = g.nodes[src];
            n.act = op.kind == XENOS_OP_RELU ? XENOS_ACT_RELU : XENOS_ACT_RELU6;
            g.node_of_tensor[n.out] = -1;
            n.out = op.out;
            n.user_ops.push_back(oi);
            g.node_of_tensor[op.out] = src;
            break;
        }
        default: {
            Node n;
            n.kind = op.kind == XENOS_OP_POOL_MAX ? NK_MAXPOOL : op.kind == XENOS_OP_POOL_AVG ? NK_AVGPOOL
                   : op.kind == XENOS_OP_POOL_GLOBAL_AVG ? NK_GAP : op.kind == XENOS_OP_ADD ? NK_ADD
                   : op.kind == XENOS_OP_MUL ? NK_MUL : op.kind == XENOS_OP_MAC ? NK_MAC
                   : op.kind == XENOS_OP_TRANSPOSE ? NK_TRANSPOSE : op.kind == XENOS_OP_SPLIT ? NK_SLICE : NK_CONCAT;
            n.in = op.in; n.out = op.out;
            n.cin = x.c; n.cout = g.tensors[op.out].c; n.k = op.k; n.stride = op.stride; n.pad = op.pad; n.act = op.act;
            n.user_ops.push_back(oi);
            g.nodes.push_back(std::move(n));
            g.node_of_tensor[op.out] = (int)g.nodes.size() - 1;
        }
        }
    }
    // every node input must be a graph input or another node's final output
    for (const Node &n : g.nodes)
        for (int t : n.in)
            if (g.tensors[t].input_slot < 0 && g.node_of_tensor[t] < 0)
                return fail(g, XENOS_E_UNSUPPORTED, "a tensor inside a fused Conv-Bn-Relu group is read by another operator");
    for (int t : g.outputs)
        if (g.node_of_tensor[t] < 0) return fail(g, XENOS_E_UNSUPPORTED, "a graph output lies inside a fused Conv-Bn-Relu group");
    return XENOS_OK;
}

// ------------------------------------------------------------------------------------------------
// Linking
// ------------------------------------------------------------------------------------------------
struct LinkCtx {
    Graph &g;
    std::vector<std::vector<int>> cons;   // tensor -> consumer node indices
    explicit LinkCtx(Graph &gg) : g(gg), cons(gg.tensors.size()) {
        for (int i = 0; i < (int)g.nodes.size(); ++i)
            for (int t : g.nodes[i].in) cons[t].push_back(i);
    }
    // the only consumer of node n's output, or -1 (graph outputs have an outside consumer)
    int sole(int n) const {
        int t = g.nodes[n].out;
        if (g.tensors[t].output_slot >= 0 || cons[t].size() != 1) return -1;
        return cons[t][0];
    }
    int rows(int n) const { const Tensor &t = g.tensors[g.nodes[n].out]; return t.h * t.w; }
};

// largest pool-output tile whose conv-output patch fits the 128-row M tile
static bool pool_patch(int k, int s, int PP, int PQ, int &th, int &tw, int &rh, int &rw) {
    int best = 0;
    for (int a = 1; a <= PP && (a - 1) * s + k <= 128; ++a)
        for (int b = 1; b <= PQ && (b - 1) * s + k <= 128; ++b) {
            int h = (a - 1) * s + k, w = (b - 1) * s + k;
            if (h * w > 128) break;
            int score = a * b;
            if (score > best || (score == best && b > tw)) { best = score; th = a; tw = b; rh = h; rw = w; }
        }
    return best > 0;
}

typedef bool (*AllowFn)(const void *, int);

// Try to grow a chain anchored at node a.  allowed(n) says whether n may join.
// Tile geometry of two linked convolutions: the producer tile rh1 x rw1 (<= 128 pixels, rw1 <= 30 so that every tap
// offset stays inside the middle buffer's spare rows) that needs the fewest tiles for a P x Q map, given the
// consumer's frame h = (k2 - 1) / 2.
static bool chain2_tile(int P, int Q, int h, int &rh1, int &rw1) {
    long best = -1;
    for (int w = 2 * h + 1; w <= std::min(Q + 2 * h, 30); ++w) {
        int hh = std::min(P + 2 * h, 128 / w);
        if (hh < 2 * h + 1) continue;
        long tiles = (long)((P + hh - 2 * h - 1) / (hh - 2 * h)) * ((Q + w - 2 * h - 1) / (w - 2 * h));
        if (best < 0 || tiles < best || (tiles == best && w > rw1)) { best = tiles; rh1 = hh; rw1 = w; }
    }
    return best > 0;
}

// Modelled time of linking two convolutions against running them one after the other (per image, arbitrary
// units): the linked form issues whole 128-row tiles for both products, frame rows included, and moves no
// intermediate; rates are what this library's kernels reach, not the device's peaks.
static bool chain2_pays(const Graph &g, const Node &A, const Node &B, bool skip) {
    const Tensor &o = g.tensors[B.out];
    const int h = (B.k - 1) / 2;
    int rh1 = 0, rw1 = 0;
    if (!chain2_tile(o.h, o.w, h, rh1, rw1)) return false;
    const double tiles = (double)((o.h + rh1 - 2 * h - 1) / (rh1 - 2 * h)) * ((o.w + rw1 - 2 * h - 1) / (rw1 - 2 * h));
    const double tc = 0.5e15, hbm = 4.0e12, px = (double)o.h * o.w;
    const double k1 = (double)A.cin * A.k * A.k, k2 = (double)A.cout * B.k * B.k;
    const double in = px * A.cin * 2, midb = px * A.cout * 2, outb = px * B.cout * 2 * (skip ? 2 : 1);
    const double lin = std::max(2.0 * tiles * 128 * (k1 * A.cout + k2 * B.cout) / tc, (in + outb) / hbm);
    const double unl = std::max(2.0 * px * k1 * A.cout / tc, (in + midb) / hbm) + std::max(2.0 * px * k2 * B.cout / tc, (midb + outb) / hbm);
    return lin <= 1.02 * unl;      // (when the model sees no difference the link still saves a launch and the bytes)
}

template <class Allowed>
static bool try_match(const LinkCtx &cx, int a, Allowed allowed, Chain &out, bool by_model = true) {
    Graph &g = cx.g;
    const Node &A = g.nodes[a];
    out = Chain();
    if (!allowed(a)) return false;
    if (g.precision == XENOS_PRECISION_FP32_CUDA_CORE) {
        // Table 1: ConvX -> ConvY -> ZPooling, with ConvY 1x1
        if (A.kind != NK_CONV) return false;
        int b = cx.sole(a);
        if (b < 0 || !allowed(b) || g.nodes[b].kind != NK_CONV) return false;
        const Node &B = g.nodes[b];
        if (B.k != 1 || B.stride != 1 || B.pad != 0) return false;
        int c = cx.sole(b);
        if (c < 0 || !allowed(c)) return false;
        const Node &C = g.nodes[c];
        if (!(C.kind == NK_MAXPOOL || C.kind == NK_AVGPOOL) || C.pad != 0) return false;
        out.kind = CK_CONV_CONV_POOL;
        out.nodes = {a, b, c};
        out.pattern = "ConvX -> ConvY -> ZPooling";
        return true;
    }
    // ---- bf16 tensor-core chains -----------------------------------------------------------
    if (A.from_matmul) {
        // MatmulX -> MatmulY (last row of Table 1) with constant right operands and nothing but a bias between
        // them: (X B1 + b1) B2 + b2 = X (B1 B2) + (b1 B2 + b2).  The constants are multiplied once at compile time
        // and the intermediate matrix never exists.  Taken only when it does not add multiplications per row.
        int b = A.act == XENOS_ACT_NONE ? cx.sole(a) : -1;
        if (b >= 0 && allowed(b) && g.nodes[b].from_matmul && g.nodes[b].kind == A.kind && A.cin % 8 == 0 &&
            (long)A.cin * g.nodes[b].cout <= (long)A.cin * A.cout + (long)A.cout * g.nodes[b].cout) {
            out.kind = CK_MATMUL_MATMUL;
            out.nodes = {a, b};
            out.pattern = "MatmulX -> MatmulY (MatA * MatB -> MatC * MatD, constants multiplied)";
            return true;
        }
    }
    if (A.kind == NK_DW) {
        // depthwise -> pointwise: the motivating mismatch of Section 2.2 (ConvX -> ConvY row)
        if (A.k != 3 || A.cin % 8 || A.stride > 2) return false;
        int b = cx.sole(a);
        if (b < 0 || !allowed(b)) return false;
        const Node &B = g.nodes[b];
        if (B.kind != NK_CONV || B.k != 1 || B.stride != 1 || B.pad != 0) return false;
        out.kind = CK_DW_PW;
        out.nodes = {a, b};
        out.pattern = "ConvX -> ConvY (depthwise 3x3 -> pointwise 1x1)";
        int c = cx.sole(b);
        const Tensor &bo = g.tensors[B.out];
        if (c >= 0 && allowed(c) && g.nodes[c].kind == NK_GAP && bo.h * ((bo.w + 3) / 4 * 4) <= 128 &&
            ((bo.h + 1) / 2) * ((bo.w + 3) / 4) <= 16) {     // whole images per tile, in 2 x 4 pixel blocks
            out.nodes.push_back(c);
            out.pattern = "ConvX -> ConvY -> ZPooling (depthwise -> pointwise -> global average)";
        }
        return true;
    }
    if (A.kind == NK_CONCAT) {
        // fire expand: {conv1x1, conv3x3} on one input, joined by channel-offset stores
        if (A.in.size() != 2) return false;
        int e0 = g.node_of_tensor[A.in[0]], e1 = g.node_of_tensor[A.in[1]];
        if (e0 < 0 || e1 < 0 || e0 == e1 || !allowed(e0) || !allowed(e1)) return false;
        const Node &E0 = g.nodes[e0], &E1 = g.nodes[e1];
        if (E0.kind != NK_CONV || E1.kind != NK_CONV || E0.in[0] != E1.in[0]) return false;
        if (cx.sole(e0) != a || cx.sole(e1) != a) return false;
        if (E0.act != E1.act || E0.stride != 1 || E1.stride != 1 || E0.cin % 8) return false;
        auto shape_ok = [](const Node &n) { return (n.k == 1 && n.pad == 0) || (n.k == 3 && n.pad == 1); };
        if (!shape_ok(E0) || !shape_ok(E1) || (E0.k == 1 && E1.k == 1)) return false;
        if (E0.cout % 8 || E1.cout % 8) return false;
        out.kind = CK_EXPAND_CONCAT;
        out.nodes = {e0, e1, a};
        out.pattern = "ConvX -> {ConvY ; ConvZ} -> concat (joined without a layout transformation)";
        {
            // the squeeze convolution in front of the two expands: its result stays in shared memory
            int sq = g.node_of_tensor[E0.in[0]];
            const std::vector<int> &sc = cx.cons[E0.in[0]];
            if (sq >= 0 && allowed(sq) && g.nodes[sq].kind == NK_CONV && !g.nodes[sq].from_matmul && g.nodes[sq].stride == 1 &&
                g.nodes[sq].cin % 64 == 0 && (g.nodes[sq].cout <= 64 || g.nodes[sq].cout % 64 == 0) && g.nodes[sq].cout <= 256 &&
                g.tensors[E0.in[0]].output_slot < 0 && sc.size() == 2 && cx.sole(a) >= -1 &&
                !(g.tensors[g.nodes[sq].in[0]].input_slot >= 0 && g.tensors[g.nodes[sq].in[0]].io_layout == XENOS_LAYOUT_NCHW)) {
                int p2 = cx.sole(a);
                const bool pooled = p2 >= 0 && g.nodes[p2].kind == NK_MAXPOOL;      // the pooled fire modules keep the pool link
                Node merged = E0.k == 3 ? E0 : E1;
                merged.cout = E0.cout + E1.cout;
                if (!pooled && (!by_model || chain2_pays(g, g.nodes[sq], merged, false))) {
                    out.kind = CK_CONV_CONV;
                    out.nodes = {sq, e0, e1, a};
                    out.pattern = "ConvX -> {ConvY ; ConvZ} -> concat, ConvX's result kept on chip (fire module)";
                    return true;
                }
            }
        }
        int p = cx.sole(a);
        if (p >= 0 && allowed(p) && g.nodes[p].kind == NK_MAXPOOL) {
            int th, tw, rh, rw;
            const Tensor &po = g.tensors[g.nodes[p].out];
            if (pool_patch(g.nodes[p].k, g.nodes[p].stride, po.h, po.w, th, tw, rh, rw)) {
                out.nodes.push_back(p);
                out.pattern += " -> ZPooling";
            }
        }
        return true;
    }
    if (A.kind == NK_CONV) {
        // a convolution that reads the caller's NCHW image stages patches of it: it links with a pool only
        const bool nchw_in = g.tensors[A.in[0]].input_slot >= 0 && g.tensors[A.in[0]].io_layout == XENOS_LAYOUT_NCHW;
        if (!nchw_in && A.cin % 8) return false;
        int b = cx.sole(a);
        if (b < 0 || !allowed(b)) return false;
        const Node &B = g.nodes[b];
        if (B.kind == NK_CONV && !nchw_in && !A.from_matmul && !B.from_matmul && A.stride == 1 && A.cin % 64 == 0 &&
            (A.cout <= 64 || A.cout % 64 == 0) && A.cout <= 256 && A.cout % 8 == 0 && B.stride == 1 &&
            ((B.k == 1 && B.pad == 0) || (B.k == 3 && B.pad == 1)) && B.cout % 8 == 0) {
            // ConvX -> ConvY (rows 1-4 of Table 1) [-> add with an identity branch]: the intermediate tile stays on chip
            int c = cx.sole(b);
            // (a 3x3 consumer that could itself feed a 1x1 convolution is left for that pairing, which needs no frame)
            if (by_model && B.k == 3 && c >= 0 && g.nodes[c].kind == NK_CONV && g.nodes[c].k == 1 && g.nodes[c].stride == 1 &&
                g.nodes[c].pad == 0 && B.cin % 64 == 0 && (B.cout <= 64 || B.cout % 64 == 0) && B.cout <= 256)
                return false;
            bool with_add = false;
            if (c >= 0 && allowed(c) && g.nodes[c].kind == NK_ADD && B.act == XENOS_ACT_NONE) {
                int other = g.nodes[c].in[0] == B.out ? g.nodes[c].in[1] : g.nodes[c].in[0];
                with_add = other != B.out;
                // a shortcut with its own 1x1 convolution is better served by the shortcut row's link (that convolution
                // joins ConvY's reduction and its result never exists): leave ConvY to it
                int pj = with_add ? g.node_of_tensor[other] : -1;
                if (by_model && pj >= 0 && pj != a && g.nodes[pj].kind == NK_CONV && g.nodes[pj].k == 1 && g.nodes[pj].pad == 0 &&
                    g.nodes[pj].act == XENOS_ACT_NONE && cx.sole(pj) == c && g.nodes[pj].chain < 0 && B.k == 1)
                    return false;
            }
            if (!by_model || chain2_pays(g, A, B, with_add)) {
                out.kind = CK_CONV_CONV;
                out.nodes = {a, b};
                out.pattern = B.k == 1 ? "ConvX -> ConvY (Conv kxk -> Conv 1x1, intermediate on chip)" : "ConvX -> ConvY (Conv kxk -> Conv 3x3, intermediate with its halo on chip)";
                if (with_add) { out.nodes.push_back(c); out.pattern += " + shortcut connection (identity)"; }
                return true;
            }
        }
        if (B.kind == NK_ADD && !nchw_in) {
            int other = B.in[0] == A.out ? B.in[1] : B.in[0];
            if (other == A.out) return false;
            out.kind = CK_CONV_TAIL;
            out.nodes = {a};
            out.pattern = "shortcut connection (ConvX -> {... -> ConvY ; identity})";
            int p = g.node_of_tensor[other];
            // the shortcut's own 1x1 convolution joins the chain as a second K segment
            if (p >= 0 && p != a && allowed(p) && g.nodes[p].kind == NK_CONV && g.nodes[p].k == 1 &&
                g.nodes[p].pad == 0 && g.nodes[p].act == XENOS_ACT_NONE && A.act == XENOS_ACT_NONE &&
                cx.sole(p) == b && g.nodes[p].cin % 8 == 0 && g.nodes[p].chain < 0) {
                out.nodes.push_back(p);
                out.pattern = "shortcut connection (ConvX -> {... -> ConvY ; ConvZ})";
            }
            out.nodes.push_back(b);
            int c = cx.sole(b);
            // (a global average is not attached to a long reduction that would run on a handful of units: the epilogue
            // with the average cannot take part in a reduction split, and at batch 1 the 72 K blocks of ResNet-18's last
            // convolution then run one after the other on 16 units, 38 us against 14 + 6 us as two kernels)
            const long gap_tiles = (long)((g.max_batch * cx.rows(b) + 127) / 128) * ((A.cout + 31) / 32);
            const bool serial_k = by_model && (long)A.k * A.k * A.cin >= 16 * 64 && gap_tiles * 2 <= g.hw.sm_count;
            if (c >= 0 && allowed(c) && g.nodes[c].kind == NK_GAP && cx.rows(b) <= 128 && !serial_k) {
                out.nodes.push_back(c);
                out.pattern += " -> ZPooling (global average)";
            }
            return true;
        }
        if (B.kind == NK_MAXPOOL) {
            int th, tw, rh, rw;
            const Tensor &po = g.tensors[B.out];
            if (!pool_patch(B.k, B.stride, po.h, po.w, th, tw, rh, rw)) return false;
            // An image convolution with its max pool is linked on request only: the pool's tiles overlap (27 % more
            // convolution rows for a 3x3 stride-2 pool) and the pooling pass of the epilogue costs what the separate pool
            // kernel costs.  Measured at batch 32, linked against the two kernels: 96 vs 77 us (7x7 stem, 64 channels),
            // 73 vs 50 us (3x3 stem, 64 channels), 166 vs 125 us (3x3, 24 channels), 830 vs 788 us (7x7 stem at 512 x 512,
            // batch 64).
            // At batch 1 the link wins (one launch less: 0.221 vs 0.231 ms for the whole 3x3-stem graph).
            // Images wider than 256 pixels keep the link: the difference is small there and the link saves the
            // convolution's output, the largest tensor of the graph (1.07 GB written and read at 512 x 512, batch 64).
            if (by_model && nchw_in && g.max_batch >= 8 && g.tensors[A.in[0]].w <= 256 && g.tensors[A.in[0]].h <= 256) return false;
            out.kind = CK_CONV_TAIL;
            out.nodes = {a, b};
            out.pattern = "ConvX -> ZPooling (CBR-MaxPooling)";
            return true;
        }
        // (an image of more than 128 pixels is averaged over several tiles when the convolution is 1x1 on 64-channel
        // blocks: its rows are then plain rows of the activation matrix)
        if (B.kind == NK_GAP && !nchw_in &&
            (cx.rows(a) <= 128 || (A.k == 1 && A.stride == 1 && A.pad == 0 && A.cin % 64 == 0 && g.precision != XENOS_PRECISION_FP32_CUDA_CORE))) {
            out.kind = CK_CONV_TAIL;
            out.nodes = {a, b};
            out.pattern = "ConvX -> ZPooling (CBR-AvgPooling, global)";
            return true;
        }
    }
    return false;
}

xenos_status_t link_pass(Graph &g) {
    LinkCtx cx(g);
    g.chains.clear();
    for (Node &n : g.nodes) n.chain = -1;
    // tensor -> node for every user tensor, including the ones folded away by the pre-fusion
    std::vector<int> node_of_any(g.tensors.size(), -1);
    for (int i = 0; i < (int)g.nodes.size(); ++i)
        for (int oi : g.nodes[i].user_ops) node_of_any[g.ops[oi].out] = i;

    auto commit = [&](Chain &c) {
        int id = (int)g.chains.size();
        for (int n : c.nodes) g.nodes[n].chain = id;
        g.chains.push_back(c);
    };
    // explicit requests first
    for (const LinkRequest &r : g.link_requests) {
        std::set<int> want;
        for (int t : r.ops) {
            int n = node_of_any[t];
            if (n < 0) return fail(g, XENOS_E_NOT_LINKABLE, "link: id is not an operator of the graph");
            if (g.nodes[n].chain >= 0) return fail(g, XENOS_E_NOT_LINKABLE, "link: operator is already part of another chain");
            want.insert(n);
        }
        bool done = false;
        for (int a : want) {
            Chain c;
            if (try_match(cx, a, [&](int n) { return want.count(n) > 0 && g.nodes[n].chain < 0; }, c, false)) {
                std::set<int> got(c.nodes.begin(), c.nodes.end());
                if (got == want) { commit(c); done = true; break; }
            }
        }
        if (!done)
            return fail(g, XENOS_E_NOT_LINKABLE,
                        "link: the requested operators match no linkable pattern that has a kernel");
    }
    if (g.link_auto) {
        // concat-anchored patterns first (their members precede the concat), then in node order
        for (int pass = 0; pass < 2; ++pass)
            for (int a = 0; a < (int)g.nodes.size(); ++a) {
                if (g.nodes[a].chain >= 0) continue;
                if ((pass == 0) != (g.nodes[a].kind == NK_CONCAT)) continue;
                Chain c;
                if (try_match(cx, a, [&](int n) { return g.nodes[n].chain < 0; }, c)) commit(c);
            }
    }
    for (int a = 0; a < (int)g.nodes.size(); ++a)
        if (g.nodes[a].chain < 0) {
            Chain c;
            c.kind = CK_SINGLE; c.nodes = {a}; c.pattern = "-";
            commit(c);
        }
    // execution order: a chain runs after the chains that produce what it reads
    int nc = (int)g.chains.size();
    std::vector<std::set<int>> deps(nc);
    for (int ci = 0; ci < nc; ++ci)
        for (int n : g.chains[ci].nodes)
            for (int t : g.nodes[n].in) {
                int p = g.node_of_tensor[t];
                if (p >= 0 && g.nodes[p].chain != ci) deps[ci].insert(g.nodes[p].chain);
            }
    std::vector<int> order, done(nc, 0);
    auto key = [&](int ci) { return *std::min_element(g.chains[ci].nodes.begin(), g.chains[ci].nodes.end()); };
    while ((int)order.size() < nc) {
        int pick = -1;
        for (int ci = 0; ci < nc; ++ci) {
            if (done[ci]) continue;
            bool ready = true;
            for (int d : deps[ci]) if (!done[d]) { ready = false; break; }
            if (ready && (pick < 0 || key(ci) < key(pick))) pick = ci;
        }
        if (pick < 0) return fail(g, XENOS_E_NOT_LINKABLE, "link: the requested chains depend on each other in a cycle");
        done[pick] = 1;
        order.push_back(pick);
    }
    std::vector<Chain> sorted;
    for (int ci : order) sorted.push_back(g.chains[ci]);
    g.chains.swap(sorted);
    for (int ci = 0; ci < nc; ++ci)
        for (int n : g.chains[ci].nodes) g.nodes[n].chain = ci;
    // attach split requests
    for (auto &rq : g.split_requests) {
        int n = node_of_any[rq.first];
        if (n < 0) return fail(g, XENOS_E_BAD_SPLIT, "split: id is not an operator of the graph");
        g.chains[g.nodes[n].chain].split = rq.second;
    }
    return XENOS_OK;
}

// ------------------------------------------------------------------------------------------------
// Split + lowering
// ------------------------------------------------------------------------------------------------
static int round_up(int v, int a) { return (v + a - 1) / a * a; }
static int ceil_div(int a, int b) { return (a + b - 1) / b; }

static size_t tensor_elems(const Tensor &t) { return t.is_vec ? (size_t)t.c : (size_t)t.c * t.h * t.w; }

struct Lower {
    Graph &g;
    explicit Lower(Graph &gg) : g(gg) {}
    int esize() const { return g.precision == XENOS_PRECISION_FP32_CUDA_CORE ? 4 : 2; }

    double tbytes(int t) const {
        const Tensor &x = g.tensors[t];
        int es = esize();
        if (g.precision == XENOS_PRECISION_BF16_TENSOR) {
            if (x.input_slot >= 0 && x.io_dtype == XENOS_DTYPE_F32) es = 4;
            if (x.output_slot >= 0 && x.is_vec) es = 4;
        }
        return (double)g.max_batch * tensor_elems(x) * es;
    }
    double node_macs(const Node &n) const {
        const Tensor &o = g.tensors[n.out];
        if (n.kind == NK_CONV) return (double)g.max_batch * o.h * o.w * n.cout * n.cin * n.k * n.k;
        if (n.kind == NK_DW) return (double)g.max_batch * o.h * o.w * n.cout * n.k * n.k;
        if (n.kind == NK_FC) return (double)g.max_batch * n.cout * n.cin;
        return 0;
    }
    double node_param_bytes(const Node &n) const {
        if (n.w.empty()) return 0;
        return (double)n.w.size() * esize() + 4.0 * n.b.size();
    }

    // ---- fp32 (CUDA-core) lowering ---------------------------------------------------------
    size_t put_f32(const std::vector<float> &v) {
        size_t off = blob_reserve(g, v.size() * 4);
        std::memcpy(g.param_blob.data() + off, v.data(), v.size() * 4);
        return off;
    }
    void push(Launch &L, int chain) {
        L.chain = chain;
        g.chains[chain].launches.push_back((int)g.launches.size());
        g.launches.push_back(L);
    }
    void fill_io(Launch &L, const Node &n) {
        const Tensor &x = g.tensors[n.in[0]];
        const Tensor &y = g.tensors[n.out];
        L.in0 = n.in[0]; L.out = n.out;
        L.C = x.c; L.H = x.h; L.W = x.w; L.K = y.c; L.P = y.h; L.Q = y.w;
        L.k = n.k; L.stride = n.stride; L.pad = n.pad; L.act = n.act;
        L.out_coff = 0; L.out_ctot = y.c;
    }
    xenos_status_t lower_single_common(int ci, int ni, bool f32) {
        const Node &n = g.nodes[ni];
        Launch L;
        L.nodes = {ni};
        fill_io(L, n);
        L.flops = 2.0 * node_macs(n);
        L.bytes = tbytes(n.out) + node_param_bytes(n);
        for (int t : n.in) L.bytes += tbytes(t);
        L.block = 256;
        switch (n.kind) {
        case NK_MAXPOOL:
        case NK_AVGPOOL:
            L.kind = f32 ? LK_F32_POOL : LK_POOL;
            L.pool_kind = n.kind == NK_MAXPOOL ? 0 : 1;
            L.pool_k = n.k; L.pool_stride = n.stride; L.pool_pad = n.pad; L.PP = L.P; L.PQ = L.Q;
            break;
        case NK_GAP:
            L.kind = f32 ? LK_F32_GAP : LK_GAP;
            L.out_dtype = (f32 || g.tensors[n.out].output_slot >= 0) ? XENOS_DTYPE_F32 : XENOS_DTYPE_BF16;
            break;
        case NK_ADD:
            L.kind = f32 ? LK_F32_ADD : LK_ADD;
            L.in1 = n.in[1];
            break;
        case NK_MUL:
        case NK_MAC:
            L.kind = f32 ? LK_F32_MULMAC : LK_MULMAC;
            L.in1 = n.in[1];
            if (n.kind == NK_MAC) L.in2 = n.in[2];
            break;
        case NK_TRANSPOSE:
            L.kind = f32 ? LK_F32_TRANSPOSE : LK_TRANSPOSE;
            if (!f32 && (L.C % 8 || L.H % 8)) return fail(g, XENOS_E_UNSUPPORTED, "bf16 transpose needs row and column counts that are multiples of 8");
            break;
        case NK_SLICE:
            L.kind = f32 ? LK_F32_SLICE : LK_SLICE;
            L.out_coff = n.pad;             // first channel of the part
            if (!f32 && (n.pad % 8 || n.cout % 8)) return fail(g, XENOS_E_UNSUPPORTED, "bf16 split needs channel offsets and counts that are multiples of 8");
            break;
        case NK_CONCAT: {
            int off = 0;
            for (int t : n.in) {
                Launch P = L;
                P.kind = f32 ? LK_F32_CONCAT_PART : LK_CONCAT_PART;
                P.in0 = t; P.C = g.tensors[t].c; P.out_coff = off; P.out_ctot = g.tensors[n.out].c;
                P.bytes = 2.0 * tbytes(t);
                off += g.tensors[t].c;
                push(P, ci);
            }
            return XENOS_OK;
        }
        default:
            return fail(g, XENOS_E_UNSUPPORTED, "internal: unexpected operator in lower_single_common");
        }
        push(L, ci);
        return XENOS_OK;
    }

    xenos_status_t lower_f32_single(int ci, int ni) {
        const Node &n = g.nodes[ni];
        if (n.kind == NK_CONV || n.kind == NK_DW || n.kind == NK_FC) {
            Launch L;
            L.nodes = {ni};
            fill_io(L, n);
            L.kind = n.kind == NK_FC ? LK_F32_FC : LK_F32_CONV;
            L.groups = n.kind == NK_DW ? n.cin : 1;
            L.w_off = put_f32(n.w); L.b_off = put_f32(n.b);
            L.flops = 2.0 * node_macs(n);
            L.bytes = tbytes(n.in[0]) + tbytes(n.out) + node_param_bytes(n);
            L.block = 256;
            if (g.chains[ci].split.user && (g.chains[ci].split.outc > 1 || g.chains[ci].split.h > 1 || g.chains[ci].split.w > 1 || g.chains[ci].split.k > 1))
                return fail(g, XENOS_E_BAD_SPLIT, "split: unlinked fp32 operators are split one output element per thread; no explicit split");
            push(L, ci);
            return XENOS_OK;
        }
        return lower_single_common(ci, ni, true);
    }

    // ConvX -> Conv1x1 -> pool as one CUDA-core kernel.  A CTA owns a tile of POOL outputs and a
    // slice of the second conv's output channels; it evaluates stage 1 on the patch the tile
    // needs (no overlap between tiles when the pool windows do not overlap).
    xenos_status_t lower_f32_linked(int ci) {
        Chain &ch = g.chains[ci];
        const Node &A = g.nodes[ch.nodes[0]], &B = g.nodes[ch.nodes[1]], &C = g.nodes[ch.nodes[2]];
        Launch L;
        L.kind = LK_F32_CONV_CONV_POOL;
        L.nodes = ch.nodes;
        fill_io(L, A);
        L.out = C.out;
        const Tensor &po = g.tensors[C.out];
        L.Cmid = A.cout; L.K2 = B.cout; L.act2 = B.act;
        L.pool_kind = C.kind == NK_MAXPOOL ? 0 : 1;
        L.pool_k = C.k; L.pool_stride = C.stride; L.pool_pad = 0; L.PP = po.h; L.PQ = po.w;
        L.out_ctot = B.cout;
        L.w_off = put_f32(A.w); L.b_off = put_f32(A.b);
        L.w2_off = put_f32(B.w); L.b2_off = put_f32(B.b);
        const SplitRequest &rq = ch.split;
        if (rq.user && rq.k > 1)
            return fail(g, XENOS_E_UNSUPPORTED, "split: the fp32 CUDA-core chain keeps every reduction inside one thread; parts_k applies to tensor-core convolutions and fc");
        const int smem_cap = std::min(g.hw.smem_bytes_per_cta, 227 * 1024) - 1024;
        auto region = [&](int t) { return (t - 1) * C.stride + C.k; };        // conv-output rows a tile of t pool rows reads
        auto smem_need = [&](int th, int tw) {
            int rh = region(th), rw = region(tw);
            int ih = (rh - 1) * A.stride + A.k, iw = (rw - 1) * A.stride + A.k;
            return (size_t)4 * ((size_t)A.cin * ih * iw + (size_t)A.cout * rh * rw);
        };
        int best_po = 0, best_th = 0, best_tw = 0;
        double best_cost = 0;
        std::vector<int> po_cands, th_cands, tw_cands;
        if (rq.user && rq.outc > 0) {
            if (rq.outc > B.cout || B.cout % rq.outc) return fail(g, XENOS_E_BAD_SPLIT, "split: parts_outc must divide the output channels");
            po_cands = {rq.outc};
        } else
            for (int p = 1; p <= B.cout && p <= 16; ++p) if (B.cout % p == 0) po_cands.push_back(p);
        auto dim_cands = [&](int req, int extent, std::vector<int> &out_tiles) -> bool {
            if (rq.user && req > 0) {
                if (req > extent) return false;
                out_tiles = {ceil_div(extent, req)};
                return ceil_div(extent, out_tiles[0]) == req;
            }
            for (int t = 1; t <= extent; ++t) out_tiles.push_back(t);
            return true;
        };
        if (!dim_cands(rq.h, po.h, th_cands)) return fail(g, XENOS_E_BAD_SPLIT, "split: parts_h does not divide the output rows into equal-height tiles");
        if (!dim_cands(rq.w, po.w, tw_cands)) return fail(g, XENOS_E_BAD_SPLIT, "split: parts_w does not divide the output columns into equal-width tiles");
        for (int p : po_cands)
            for (int th : th_cands)
                for (int tw : tw_cands) {
                    if (smem_need(th, tw) > (size_t)smem_cap) continue;
                    int ctas = p * ceil_div(po.h, th) * ceil_div(po.w, tw);
                    double s1 = (double)region(th) * region(tw) * A.cout * A.cin * A.k * A.k;
                    double s2 = (double)region(th) * region(tw) * (B.cout / p) * A.cout;
                    // modelled time: waves over the units, plus a fixed per-CTA overhead worth 2048 MACs
                    double cost = (double)ceil_div(ctas * g.max_batch, g.hw.sm_count) * (s1 + s2 + 2048.0);
                    if (best_po == 0 || cost < best_cost) { best_cost = cost; best_po = p; best_th = th; best_tw = tw; }
                }
        if (best_po == 0) return fail(g, XENOS_E_BAD_SPLIT, "split: no tile of the linked chain fits shared memory");
        L.parts_outc = best_po; L.tile_h = best_th; L.tile_w = best_tw;
        L.tiles_h = ceil_div(po.h, best_th); L.tiles_w = ceil_div(po.w, best_tw);
        L.halo_h = region(best_th); L.halo_w = region(best_tw);
        L.smem_bytes = (int)smem_need(best_th, best_tw);
        L.grid = L.parts_outc * L.tiles_h * L.tiles_w;   // per image
        L.block = 128;
        L.flops = 2.0 * (node_macs(A) + node_macs(B));
        L.bytes = tbytes(A.in[0]) + tbytes(C.out) + node_param_bytes(A) + node_param_bytes(B);
        push(L, ci);
        return XENOS_OK;
    }

    // ---- bf16 tensor-core lowering ---------------------------------------------------------
    // Packs the [npad][kpad] bf16 weight matrix of an implicit GEMM: row n = output channel,
    // K order = (tap r*k+s, input channel c) per segment, each segment padded to 64.
    struct WSrc { const Node *n; int row0; int seg; bool centre_only; };

    xenos_status_t make_gemm(int ci, const std::vector<int> &cover, const Node *dw, const Node *mainc,
                             const Node *shortcut, const Node *expand2, const Node *addn, const Node *pooln,
                             const Node *gapn, const Node *catn, bool fc) {
        Chain &ch = g.chains[ci];
        Launch L;
        L.kind = LK_GEMM;
        L.nodes = cover;
        const Node &M = *mainc;
        const Tensor &src = g.tensors[dw ? dw->in[0] : M.in[0]];
        const Tensor &convout = g.tensors[M.out];
        L.in0 = dw ? dw->in[0] : M.in[0];
        L.C = src.c; L.H = fc ? 1 : src.h; L.W = fc ? 1 : src.w;
        L.P = fc ? 1 : convout.h; L.Q = fc ? 1 : convout.w;
        L.rows_per_image = L.P * L.Q;
        L.k = M.k; L.stride = M.stride; L.pad = M.pad;
        int N = M.cout + (expand2 ? expand2->cout : 0);
        L.K = N;
        // --- A segments
        ASeg &s0 = L.seg[0];
        s0.tensor = L.in0; s0.C = src.c; s0.H = L.H; s0.W = L.W;
        int kk = expand2 ? std::max(M.k, expand2->k) : M.k;     // merged expand reads the 3x3 window
        int kpadg = expand2 ? 1 : M.pad;
        if (dw) {
            s0.mode = AM_DW; s0.k = dw->k; s0.stride = dw->stride; s0.pad = dw->pad;
            s0.kelems = src.c; s0.dw_act = dw->act;
            // depthwise taps, tap-major fp32 [9][C], so a thread reads 8 consecutive channels per tap
            std::vector<float> wt((size_t)9 * src.c);
            for (int c = 0; c < src.c; ++c)
                for (int t = 0; t < 9; ++t) wt[(size_t)t * src.c + c] = dw->w[(size_t)c * 9 + t];
            s0.dw_w_off = put_f32(wt);
            s0.dw_b_off = put_f32(dw->b);
        } else if (src.input_slot >= 0 && src.io_layout == XENOS_LAYOUT_NCHW) {
            if (expand2) return fail(g, XENOS_E_UNSUPPORTED, "internal: expand on an NCHW input");
            // K order of a stem with k > 4: (channel, tap row) segments of 8 elements, the taps of one window row,
            // which are adjacent in the image: a producer thread copies a segment instead of gathering elements.
            // Small kernels keep (tap, channel) order without padding inside K.
            if (M.k > 8) return fail(g, XENOS_E_UNSUPPORTED, "a convolution on an NCHW image supports kernels up to 8 x 8");
            s0.mode = AM_STEM; s0.k = M.k; s0.stride = M.stride; s0.pad = M.pad;
            s0.kelems = M.k > 4 ? src.c * M.k * 8 : M.k * M.k * src.c; s0.src_dtype = src.io_dtype;
        } else {
            if (src.c % 8) return fail(g, XENOS_E_UNSUPPORTED, "bf16 NHWC tensors need a channel count that is a multiple of 8");
            s0.mode = AM_GATHER; s0.k = kk; s0.stride = M.stride; s0.pad = expand2 ? kpadg : M.pad;
            s0.kelems = kk * kk * src.c;
        }
        s0.kblocks = ceil_div(s0.kelems, 64);
        ASeg &s1 = L.seg[1];
        if (shortcut) {
            const Tensor &ss = g.tensors[shortcut->in[0]];
            s1.mode = AM_GATHER; s1.tensor = shortcut->in[0]; s1.C = ss.c; s1.H = ss.h; s1.W = ss.w;
            s1.k = 1; s1.stride = shortcut->stride; s1.pad = 0; s1.kelems = ss.c; s1.kblocks = ceil_div(ss.c, 64);
        }
        L.kblocks = s0.kblocks + s1.kblocks;
        L.kpad = 64 * L.kblocks;
        // --- epilogue
        L.act = M.act;
        const Node *last = mainc;
        if (catn) last = catn;
        if (addn) {
            last = addn;
            L.act2 = addn->act;
            if (!shortcut) L.skip = addn->in[0] == M.out ? addn->in[1] : addn->in[0];
        }
        if (pooln) {
            last = pooln;
            L.epi = EPI_POOL; L.map_mode = MAP_PATCH;
            L.pool_kind = 0; L.pool_k = pooln->k; L.pool_stride = pooln->stride; L.pool_pad = pooln->pad;
            const Tensor &po = g.tensors[pooln->out];
            L.PP = po.h; L.PQ = po.w;
            if (!pool_patch(pooln->k, pooln->stride, po.h, po.w, L.patch_th, L.patch_tw, L.patch_rh, L.patch_rw))
                return fail(g, XENOS_E_UNSUPPORTED, "internal: pool patch does not fit");
            L.tiles_y = ceil_div(po.h, L.patch_th); L.tiles_x = ceil_div(po.w, L.patch_tw);
            L.ni = 1;
            L.step_y = L.patch_th * pooln->stride; L.step_x = L.patch_tw * pooln->stride;
            L.off_y = L.off_x = pooln->pad;
            L.tile_rows = L.patch_rh * L.patch_rw;
        }
        if (gapn) {
            last = gapn;
            L.epi = EPI_GAP;
            L.imgs_per_tile = 128 / L.rows_per_image;
            L.tile_rows = L.imgs_per_tile * L.rows_per_image;
            L.gap_imgs = L.imgs_per_tile; L.gap_area = L.rows_per_image; L.gap_rpi = L.rows_per_image;
            if (L.rows_per_image > 128) {
                // several tiles per image: 128 rows each, their column sums combined by the tile that finishes last
                if (dw || shortcut || expand2 || M.k != 1 || M.stride != 1 || M.pad != 0 || src.c % 64)
                    return fail(g, XENOS_E_UNSUPPORTED, "internal: global average over more than 128 pixels needs a 1x1 convolution on 64-channel blocks");
                L.gap_parts = ceil_div(L.rows_per_image, 128);
                L.imgs_per_tile = 1; L.tile_rows = 128;
                L.gap_imgs = 1; L.gap_area = 128;
            }
        }
        // Where a 64-channel K block of the activation operand is a box of the NHWC tensor (stride 1, channels a
        // multiple of 64, no second K segment), TMA fetches it and writes the operand layout itself: the rows of
        // the [pixels][C] matrix for a 1x1 convolution or fc, the tile's patch shifted by the tap for k x k.
        if (s0.mode == AM_GATHER && !expand2 && !shortcut && !pooln && src.c % 64 == 0 && M.stride == 1) {
            if (M.k == 1 && M.pad == 0) {
                L.a_tma = 1;
                L.a_box_bytes = 128 * 128;
            } else if (!gapn && !fc) {
                // patch tiles: ni whole images when one fits 128 rows, else rh x rw output pixels with the fewest tiles
                L.a_tma = 2;
                L.map_mode = MAP_PATCH;
                if (L.P * L.Q <= 128) {
                    L.patch_rh = L.P; L.patch_rw = L.Q; L.ni = std::min(128 / (L.P * L.Q), g.max_batch);
                    // (fewer images per tile while units would idle, as for the depthwise chains)
                    while (L.ni > 1 && (long)ceil_div(g.max_batch, L.ni) * ceil_div(round_up(N, 16), 256) * 2 <= g.hw.sm_count) --L.ni;
                } else {
                    L.ni = 1;
                    long best = -1;
                    for (int tw = 1; tw <= std::min(L.Q, 128); ++tw) {
                        int th = std::min(L.P, 128 / tw);
                        long tiles = (long)ceil_div(L.P, th) * ceil_div(L.Q, tw);
                        if (best < 0 || tiles < best || (tiles == best && tw > L.patch_rw)) { best = tiles; L.patch_rh = th; L.patch_rw = tw; }
                    }
                }
                L.tiles_y = ceil_div(L.P, L.patch_rh); L.tiles_x = ceil_div(L.Q, L.patch_rw);
                L.step_y = L.patch_rh; L.step_x = L.patch_rw; L.off_y = L.off_x = 0;
                L.tile_rows = L.ni * L.patch_rh * L.patch_rw;
                L.a_box_bytes = L.tile_rows * 128;
            }
        }
        if (s0.mode == AM_STEM) {
            // The stem stages the tile's input patch in shared memory, so its tile is a patch too:
            // the pool patch when a pool is linked, else th x tw output pixels with the fewest tiles.
            if (gapn) return fail(g, XENOS_E_UNSUPPORTED, "a convolution on an NCHW image cannot be linked with a global average");
            if (!pooln) {
                L.map_mode = MAP_PATCH;
                L.ni = 1;
                long best = -1;
                for (int tw = 1; tw <= std::min(L.Q, 128); ++tw) {
                    int th = std::min(L.P, 128 / tw);
                    // (tiles whose input patch the copy engine can fetch: at most 256 columns and rows)
                    if (tw > 1 && ((tw - 1) * M.stride + (M.k > 4 ? 10 : M.k) + 8 > 256 || (th - 1) * M.stride + M.k > 256)) continue;
                    long tiles = (long)ceil_div(L.P, th) * ceil_div(L.Q, tw);
                    if (best < 0 || tiles < best || (tiles == best && tw > L.patch_rw)) { best = tiles; L.patch_rh = th; L.patch_rw = tw; }
                }
                L.tiles_y = ceil_div(L.P, L.patch_rh); L.tiles_x = ceil_div(L.Q, L.patch_rw);
                L.step_y = L.patch_rh; L.step_x = L.patch_rw; L.off_y = L.off_x = 0;
                L.tile_rows = L.patch_rh * L.patch_rw;
            }
            // TMA fetches the patch when the image rows are 16-byte multiples; the box is widened so
            // that its x origin can be rounded down to a 16-byte boundary
            const int es = src.io_dtype == XENOS_DTYPE_F32 ? 4 : 2;
            L.stem_align = 16 / es;
            L.stem_tma = (src.w * es) % 16 == 0 ? 1 : 0;
            L.halo_h = (L.patch_rh - 1) * M.stride + M.k;
            // (a segment is read whole, kp elements plus up to two for the alignment of 16-bit images)
            L.halo_w = round_up((L.patch_rw - 1) * M.stride + (M.k > 4 ? 8 + 2 : M.k) + L.stem_align - 1, L.stem_align);
            L.halo_cb = src.c;
            // (small kernels keep patch offsets as 16-bit table entries)
            if (L.halo_h > 256 || L.halo_w > 256 || src.c > 256 || (M.k <= 4 && (long)src.c * L.halo_h * L.halo_w >= 65535)) L.stem_tma = 0;
            if (L.stem_tma) {
                L.halo_bytes = src.c * L.halo_h * L.halo_w * es;
                L.halo_stride = (int)align_up((size_t)L.halo_bytes, 128);
            }
        }
        if (dw) {
            // The depthwise stage reads a halo tile that TMA fetches as one 4-D box, so the tile is a
            // patch: ni whole images when an image fits 128 rows, else th x tw output pixels of one image.
            L.map_mode = MAP_PATCH;
            // the tile's row pitch is a multiple of 4: a producer thread owns 4 adjacent pixels of a row
            // ... made of br x 4 pixel blocks, the unit of work of a depthwise producer thread: 16 blocks of
            // 2 x 4 when a K block has 64 channels, 32 blocks of 1 x 4 otherwise
            const int Qp = round_up(L.Q, 4);
            const int br = std::min(64, src.c) > 32 ? 2 : 1, nblk = br == 2 ? 16 : 32;
            auto blocks_of = [&](int th, int tw) { return ceil_div(th, br) * (tw / 4); };
            if (L.P * Qp <= 128 && blocks_of(L.P, Qp) <= nblk) {
                L.ni = std::min(128 / (L.P * Qp), nblk / blocks_of(L.P, Qp)); L.patch_rh = L.P; L.patch_rw = Qp;
            } else {
                if (gapn) return fail(g, XENOS_E_UNSUPPORTED, "internal: global average needs whole images per tile");
                L.ni = 1;
                long best = -1;
                for (int tw = 4; tw <= std::min(Qp, 64); tw += 4) {
                    int th = std::min(L.P, br * (nblk / (tw / 4)));
                    long tiles = (long)ceil_div(L.P, th) * ceil_div(L.Q, tw);
                    // fewest tiles first; then the widest tile (longest contiguous rows in memory)
                    if (best < 0 || tiles < best || (tiles == best && tw > L.patch_rw)) { best = tiles; L.patch_rh = th; L.patch_rw = tw; }
                }
            }
            // keep one halo tile (64 channels of the input window) small enough for a 2-3 deep ring
            auto halo_of = [&](int ni, int th, int tw) {
                return (long)ni * ((round_up(th, br) - 1) * dw->stride + 3) * ((tw - 1) * dw->stride + 3) * std::min(64, src.c) * 2;
            };
            while (L.ni > 1 && halo_of(L.ni, L.patch_rh, L.patch_rw) > 40 * 1024) --L.ni;
            // the depthwise stage is recomputed per channel tile and its time grows with the tile's pixels:
            // while SMs would stay idle, fewer images per tile spread it over more of them
            while (L.ni > 1 && (long)ceil_div(g.max_batch, L.ni) * ceil_div(round_up(N, 16), 256) * 2 <= g.hw.sm_count) --L.ni;
            while (!gapn && L.patch_rh > 1 && halo_of(L.ni, L.patch_rh, L.patch_rw) > 76 * 1024) --L.patch_rh;
            // Small batches leave most units idle while each tile's depthwise stage runs its K blocks one after the
            // other, at a pace set by the pixels per tile: while at least half of the units would stay idle, halve the
            // tile's rows (the MMA tile is then partly empty, which costs nothing there).
            while (!gapn && L.ni == 1 && L.patch_rh > 1 &&
                   (long)g.max_batch * ceil_div(L.P, (L.patch_rh + 1) / 2) * ceil_div(L.Q, L.patch_rw) * ceil_div(round_up(N, 16), 256) * 2 <= g.hw.sm_count)
                L.patch_rh = (L.patch_rh + 1) / 2;
            L.tiles_y = ceil_div(L.P, L.patch_rh); L.tiles_x = ceil_div(L.Q, L.patch_rw);
            L.step_y = L.patch_rh; L.step_x = L.patch_rw; L.off_y = L.off_x = 0;
            L.tile_rows = L.ni * L.patch_rh * L.patch_rw;
            // (the box covers whole blocks: a producer thread reads its block's full window)
            L.halo_h = (round_up(L.patch_rh, br) - 1) * dw->stride + 3; L.halo_w = (L.patch_rw - 1) * dw->stride + 3;
            L.halo_cb = std::min(64, src.c);
            L.halo_bytes = L.ni * L.halo_h * L.halo_w * L.halo_cb * 2;
            L.halo_stride = (int)align_up((size_t)L.halo_bytes, 128);
            if (L.halo_h > 256 || L.halo_w > 256) return fail(g, XENOS_E_UNSUPPORTED, "internal: halo tile exceeds the TMA box limit");
            if (gapn) { L.gap_imgs = L.ni; L.gap_area = L.patch_rh * L.patch_rw; L.gap_rpi = L.rows_per_image; }
        }
        L.out = last->out;
        const Tensor &ot = g.tensors[L.out];
        L.out_ctot = ot.c; L.out_coff = 0;
        L.out_dtype = (ot.is_vec && ot.output_slot >= 0) ? XENOS_DTYPE_F32 : XENOS_DTYPE_BF16;
        if (!ot.is_vec && ot.c % 8) return fail(g, XENOS_E_UNSUPPORTED, "bf16 NHWC tensors need a channel count that is a multiple of 8");
        // --- split (Section 4.2.1: output channels first, then rows / columns of the feature map)
        const SplitRequest &rq = ch.split;
        int N16 = round_up(N, 16);
        if (L.map_mode == MAP_PATCH) L.m_tiles = ceil_div(g.max_batch, L.ni) * L.tiles_y * L.tiles_x;
        else if (L.epi == EPI_GAP) L.m_tiles = L.gap_parts > 1 ? g.max_batch * L.gap_parts : ceil_div(g.max_batch, L.imgs_per_tile);
        else L.m_tiles = ceil_div(g.max_batch * L.rows_per_image, 128);
        if (rq.user && (rq.h > 1 || rq.w > 1))
            return fail(g, XENOS_E_BAD_SPLIT, "split: tensor-core chains cut rows / columns into 128-row tiles themselves; only parts_outc can be set");
        if (rq.user && rq.outc > 0) {
            L.n_tiles = rq.outc;
            L.tile_n = round_up(ceil_div(N16, rq.outc), 16);
            if (L.tile_n > 256 || (rq.outc - 1) * L.tile_n >= N)
                return fail(g, XENOS_E_BAD_SPLIT, "split: parts_outc gives an output-channel tile that is empty or wider than 256");
        } else {
            L.n_tiles = ceil_div(N16, 256);
            L.tile_n = round_up(ceil_div(N16, L.n_tiles), 16);
            // kernels are dealt to idle units first: halve the channel tile while units stay idle
            // (a linked depthwise stage is recomputed per channel tile, so it stops halving earlier)
            // (unless most units are idle anyway: then narrower channel tiles shorten every CTA's weight loads and store)
            const int min_tile_n = dw ? ((long)L.m_tiles * L.n_tiles * 4 <= g.hw.sm_count ? 64 : 256) : 32;
            while (L.m_tiles * L.n_tiles < g.hw.sm_count && L.tile_n >= 2 * min_tile_n) {
                int nt = L.n_tiles * 2, tn = round_up(ceil_div(N16, nt), 16);
                if ((nt - 1) * tn >= N) break;
                L.n_tiles = nt; L.tile_n = tn;
            }
        }
        L.npad = L.n_tiles * L.tile_n;
        // --- reduction split (Section 4.2.2: C, R, S after K; it needs an additional reduction).  The K blocks
        // (64 elements of the (tap, channel) order) are cut into chunks of equal size, ascending; a chunk's partial
        // sums are fp32 and the chunks are added in ascending order.  Chosen automatically only when the tiles
        // leave most units idle and K is long (fc, late convolutions at small batch).
        {
            // (a linked depthwise stage can be split on request: a chunk's CTA then produces only its own channels of
            // the depthwise result.  It is not chosen automatically: measured at batch 1 the partial sums and their
            // reduction cost more than the shorter depthwise loop saves; the split search may still pick it.)
            // (a fully connected layer of at most 8 vectors runs on the CUDA cores: one pass over the weight matrix,
            // no partial sums; its input must be a bf16 vector that fits shared memory.  Measured, 1024 -> 1000:
            // 6.6 against 12 us at batch 1, 16.8 against 15.8 us at batch 32, where the tensor-core tiles win)
            if (fc && !rq.user && g.max_batch <= 8 && L.epi == EPI_STORE && L.skip < 0 && !shortcut && src.c % 8 == 0 &&
                (long)g.max_batch * src.c * 2 <= 160 * 1024 && !(src.input_slot >= 0 && src.io_dtype != XENOS_DTYPE_BF16))
                L.fc_small = 1;
            const bool plain = !L.fc_small && s0.mode == AM_GATHER && (L.map_mode == MAP_FLAT || L.a_tma == 2);
            // (a linked shortcut convolution, the second K segment of a gathered convolution, is cut with it: the chunks
            // are blocks of the concatenated K)
            const bool can = ((plain || s0.mode == AM_DW) && s1.mode == AM_NONE && L.epi == EPI_STORE) ||
                             (plain && L.map_mode == MAP_FLAT && !L.a_tma && s1.mode == AM_GATHER && L.epi == EPI_STORE);
            int want = 1;
            if (rq.user && rq.k > 1) {
                if (!can) return fail(g, XENOS_E_UNSUPPORTED, "split: parts_k applies to a convolution, depthwise -> pointwise chain or fc that stores its tile (no image stem or pooling epilogue)");
                if (rq.k > L.kblocks) return fail(g, XENOS_E_BAD_SPLIT, "split: parts_k exceeds the number of 64-element K blocks");
                want = rq.k;
            } else if (!rq.user && can && plain && L.kblocks >= 4 && (long)L.m_tiles * L.n_tiles * 2 <= g.hw.sm_count) {
                want = std::min(L.kblocks / 2, g.hw.sm_count / (L.m_tiles * L.n_tiles));
            }
            if (want > 1) {
                L.kb_per = ceil_div(L.kblocks, want);
                L.ksplit = ceil_div(L.kblocks, L.kb_per);
                if (rq.user && rq.k > 1 && L.ksplit != want)
                    return fail(g, XENOS_E_BAD_SPLIT, "split: parts_k does not cut the K blocks into that many non-empty chunks of equal size");
                if (L.ksplit < 2) { L.ksplit = 1; L.kb_per = 0; }
            }
        }
        // A depthwise -> pointwise chain with at most one tile per CTA and two 256-wide channel tiles: one CTA keeps both
        // channel tiles of its pixels (the two accumulators hold one 512-column tile; with a single tile per CTA
        // nothing is double-buffered anyway), so the depthwise stage is computed once per pixel tile instead of once
        // per channel tile, and the tiles get fewer rows until they cover the units again.
        if (dw && L.epi == EPI_STORE && L.ksplit == 1 && s1.mode == AM_NONE && !rq.user && L.ni == 1 && L.tile_n == 256 &&
            L.n_tiles % 2 == 0 && L.halo_cb == 64 && (long)L.m_tiles * L.n_tiles <= g.hw.sm_count) {
            const int nt2 = L.n_tiles / 2;
            int th = L.patch_rh;
            for (int t = 1; t <= L.patch_rh; ++t)
                if ((long)g.max_batch * ceil_div(L.P, t) * L.tiles_x * nt2 <= g.hw.sm_count) { th = t; break; }
            const int hh = (th - 1) * dw->stride + 3;
            const int hstride = (int)align_up((size_t)hh * L.halo_w * 128, 128);
            const int room2 = std::min(g.hw.smem_bytes_per_cta, 227 * 1024) - 1024 - 256 - 2048 - (int)align_up((size_t)40 * src.c, 128);
            if (2 * (16384 + 2 * 256 * 128) + 2 * hstride <= room2) {
                L.n_acc = 2; L.n_tiles = nt2;
                L.patch_rh = th; L.tiles_y = ceil_div(L.P, th); L.step_y = th;
                L.tile_rows = th * L.patch_rw;
                L.halo_h = hh; L.halo_bytes = hh * L.halo_w * 128; L.halo_stride = hstride;
                L.m_tiles = g.max_batch * L.tiles_y * L.tiles_x;
            }
        }
        // two accumulators in tensor memory so the epilogue of one tile overlaps the MMAs of the next
        L.acc_stride = round_up(L.tile_n, 32);
        L.tmem_cols = 32;
        while (L.tmem_cols < 2 * L.acc_stride) L.tmem_cols *= 2;
        if (L.tmem_cols > g.hw.tmem_columns) return fail(g, XENOS_E_BAD_SPLIT, "split: accumulator tiles exceed tensor memory columns");
        // shared memory of the one persistent CTA per SM: [A|B ring][halo ring][epilogue staging][barriers]
        int stage_bytes = 16384 + L.n_acc * L.tile_n * 128;
        int stg_bytes = L.epi == EPI_POOL ? 128 * (L.tile_n * 2 + 16) : (L.epi == EPI_GAP ? 128 * 33 * 4 + 512 : 0);
        stg_bytes = (int)align_up((size_t)stg_bytes, 128);
        // depthwise tap weights + bias of the linked stage (fp32 [10][C]) and two bias slices of the GEMM
        // (a TMA-fed stem keeps its K-index -> patch-offset table there instead)
        int dww_bytes = dw ? (int)align_up((size_t)40 * src.c, 128) : (L.stem_tma ? (int)align_up((size_t)L.kpad * 2, 128) : 0);
        int cap = std::min(g.hw.smem_bytes_per_cta, 227 * 1024) - 1024 - 256 - 2048 - dww_bytes;
        // a linked depthwise stage is bound by its own arithmetic, not by the MMA: give the halo ring
        // (the TMA prefetch distance) up to four stages first, the A|B ring keeps three when it can
        L.hstages = 0;
        if (dw || L.stem_tma) {
            L.hstages = 2;
            while (L.hstages < 4 && cap - stg_bytes - (L.hstages + 1) * L.halo_stride >= 3 * stage_bytes) ++L.hstages;
        }
        int room = cap - stg_bytes - L.hstages * L.halo_stride;
        L.stages = std::min(6, room / stage_bytes);
        if (L.stages < 1) return fail(g, XENOS_E_BAD_SPLIT, "split: pipeline does not fit shared memory");
        L.off_halo = L.stages * stage_bytes;
        L.off_stg = L.off_halo + L.hstages * L.halo_stride;
        L.off_dww = (int)align_up((size_t)(L.off_stg + stg_bytes), 128);
        L.off_bias = L.off_dww + dww_bytes;
        L.off_bar = L.off_bias + 2048;
        L.pipe_bytes = L.off_bar;
        L.smem_bytes = L.off_bar + 256 + 1024;     // + barriers, alignment slack
        L.grid = std::min(L.m_tiles * L.n_tiles * L.ksplit, g.hw.sm_count);
        L.block = 448;
        // A depthwise -> pointwise chain that stores its tile and has one tile per CTA at most runs in the kernel whose
        // warps all work on the stencil and then on the store (dwpw_kernel: 16 worker warps for 64-channel blocks, 8
        // for narrower ones): with a single tile the separate producer and epilogue warps of gemm_chain_kernel
        // would take turns waiting.  Measured on MobileNet at batch 32: 18.8 against 20.1 us per 14 x 14 chain; the
        // chains with many tiles per CTA are faster in gemm_chain_kernel (44 against 48 us for the first one).
        // (a global-average epilogue parks its slabs in the A|B ring, which a CTA's only tile has left free)
        const int gap_workers = L.halo_cb > 32 ? 16 : 8;
        const long gap_need = (long)(gap_workers / 4) * 128 * 33 * 4 + 4L * std::max(32 * gap_workers, (gap_workers / 4) * L.gap_imgs * 32);
        const bool gap_fits = L.epi == EPI_GAP && L.skip < 0 && L.act2 == 0 && (long)L.stages * stage_bytes >= gap_need;
        if (dw && (L.epi == EPI_STORE || gap_fits) && L.ksplit == 1 && s1.mode == AM_NONE && L.m_tiles * L.n_tiles <= g.hw.sm_count) {
            L.dw_workers = L.halo_cb > 32 ? 16 : 8;
            L.block = 64 + 32 * L.dw_workers;
        }
        // --- pack weights + bias
        L.w_off = blob_reserve(g, (size_t)L.npad * L.kpad * 2);
        L.b_off = blob_reserve(g, (size_t)L.npad * 4);
        uint16_t *wp = reinterpret_cast<uint16_t *>(g.param_blob.data() + L.w_off);
        float *bp = reinterpret_cast<float *>(g.param_blob.data() + L.b_off);
        auto pack_conv = [&](const Node &n, int row0, int kbase, int kwin, int C) {
            // n.w is [cout][C][n.k][n.k]; it sits centred in a kwin x kwin window
            int shift = (kwin - n.k) / 2;
            for (int o = 0; o < n.cout; ++o)
                for (int c = 0; c < C; ++c)
                    for (int r = 0; r < n.k; ++r)
                        for (int s = 0; s < n.k; ++s) {
                            int tap = (r + shift) * kwin + (s + shift);
                            wp[(size_t)(row0 + o) * L.kpad + kbase + tap * C + c] =
                                f32_to_bf16_rne(n.w[(((size_t)o * C + c) * n.k + r) * n.k + s]);
                        }
            for (int o = 0; o < n.cout; ++o) bp[row0 + o] += n.b[o];
        };
        if (fc || dw) {
            for (int o = 0; o < M.cout; ++o) {
                for (int c = 0; c < M.cin; ++c) wp[(size_t)o * L.kpad + c] = f32_to_bf16_rne(M.w[(size_t)o * M.cin + c]);
                bp[o] = M.b[o];
            }
        } else if (expand2) {
            // concat order decides the row offsets; both read the same kk x kk window
            pack_conv(M, 0, 0, kk, src.c);
            pack_conv(*expand2, M.cout, 0, kk, src.c);
        } else if (s0.mode == AM_STEM && M.k > 4) {
            const int kp = 8;
            for (int o = 0; o < M.cout; ++o) {
                for (int c = 0; c < src.c; ++c)
                    for (int r = 0; r < M.k; ++r)
                        for (int sx = 0; sx < M.k; ++sx)
                            wp[(size_t)o * L.kpad + (c * M.k + r) * kp + sx] =
                                f32_to_bf16_rne(M.w[(((size_t)o * src.c + c) * M.k + r) * M.k + sx]);
                bp[o] += M.b[o];
            }
        } else {
            pack_conv(M, 0, 0, M.k, src.c);
        }
        if (shortcut) pack_conv(*shortcut, 0, 64 * s0.kblocks, 1, s1.C);
        // --- modelled work
        for (int ni : cover) L.flops += 2.0 * node_macs(g.nodes[ni]);
        L.bytes = tbytes(L.in0) + tbytes(L.out) + (double)L.npad * L.kpad * 2 + 4.0 * L.npad;
        if (shortcut) L.bytes += tbytes(s1.tensor);
        if (L.skip >= 0) L.bytes += tbytes(L.skip);
        if (dw) L.bytes += node_param_bytes(*dw);
        push(L, ci);
        return XENOS_OK;
    }

    // ---- two linked convolutions, intermediate tile in shared memory (chain2_kernel) ---------------------------
    // A: first convolution (stride 1, input channels a multiple of 64).  Second stage: one convolution B (1x1, or
    // 3x3 with padding 1), or the two expand convolutions of a fire module merged over the 3x3 window in concat order.
    xenos_status_t make_gemm2(int ci, const std::vector<int> &cover, const Node &A, const Node *B, const Node *E0, const Node *E1,
                              const Node *addn, const Node *last) {
        Launch L;
        L.kind = LK_GEMM2;
        L.nodes = cover;
        const Tensor &src = g.tensors[A.in[0]];
        const Tensor &ot = g.tensors[last->out];
        const int k2 = B ? B->k : 3, h = (k2 - 1) / 2;
        const int N2 = B ? B->cout : E0->cout + E1->cout;
        L.in0 = A.in[0]; L.out = last->out;
        L.C = src.c; L.H = src.h; L.W = src.w; L.P = ot.h; L.Q = ot.w; L.K = N2; L.rows_per_image = L.P * L.Q;
        L.k = A.k; L.stride = 1; L.pad = A.pad; L.k2 = k2; L.halo2 = h;
        L.Cmid = A.cout; L.n1pad = round_up(A.cout, 64);
        L.seg[0].tensor = L.in0; L.seg[0].C = src.c; L.seg[0].H = src.h; L.seg[0].W = src.w; L.seg[0].k = A.k; L.seg[0].pad = A.pad;
        L.kblocks = A.k * A.k * (src.c / 64);
        L.kblocks2 = k2 * k2 * (L.n1pad / 64);
        L.act = A.act; L.act2 = B ? B->act : E0->act;
        if (addn) {
            L.act3 = addn->act;
            const int mine = B->out;
            L.skip = addn->in[0] == mine ? addn->in[1] : addn->in[0];
        }
        if (src.c % 64 || g.tensors[A.out].h != ot.h || g.tensors[A.out].w != ot.w)
            return fail(g, XENOS_E_UNSUPPORTED, "internal: two linked convolutions need 64-channel input blocks and a consumer of equal extent");
        if (!chain2_tile(L.P, L.Q, h, L.patch_rh, L.patch_rw)) return fail(g, XENOS_E_UNSUPPORTED, "internal: no tile for two linked convolutions");
        L.rh2 = L.patch_rh - 2 * h; L.rw2 = L.patch_rw - 2 * h;
        L.tiles_y = ceil_div(L.P, L.rh2); L.tiles_x = ceil_div(L.Q, L.rw2);
        L.m_tiles = g.max_batch * L.tiles_y * L.tiles_x;
        L.a_box_bytes = L.patch_rh * L.patch_rw * 128;
        const int N216 = round_up(N2, 16);
        L.n_tiles = ceil_div(N216, 256);
        L.tile_n = round_up(ceil_div(N216, L.n_tiles), 16);
        L.npad = L.n_tiles * L.tile_n;
        L.out_ctot = ot.c; L.out_coff = 0;
        L.stage_bytes = 16384 + std::max(L.n1pad, L.tile_n) * 128;
        const int mid_bytes = (L.n1pad / 64) * (128 + 64) * 128;
        const int cap = std::min(g.hw.smem_bytes_per_cta, 227 * 1024) - 1024 - 256;
        L.stages = std::min(6, (cap - mid_bytes) / L.stage_bytes);
        if (L.stages < 2) return fail(g, XENOS_E_BAD_SPLIT, "split: two linked convolutions do not fit shared memory");
        L.off_mid = L.stages * L.stage_bytes;
        L.off_bar = L.off_mid + mid_bytes;
        L.smem_bytes = L.off_bar + 256 + 1024;
        L.tmem_cols = 512;
        L.grid = std::min(L.m_tiles, g.hw.sm_count);
        L.block = 320;
        if (g.chains[ci].split.user && (g.chains[ci].split.outc > 1 || g.chains[ci].split.h > 1 || g.chains[ci].split.w > 1 || g.chains[ci].split.k > 1))
            return fail(g, XENOS_E_BAD_SPLIT, "split: two linked convolutions keep all output channels of a tile in one CTA; no explicit split");
        // --- parameters: W1 [n1pad][K1], bias1 [n1pad]; W2 [npad][k2*k2*n1pad], bias2 [npad]; K order (tap, channel)
        const int K1 = L.kblocks * 64, K2 = L.kblocks2 * 64;
        L.kpad = K1;
        L.w_off = blob_reserve(g, (size_t)L.n1pad * K1 * 2);
        L.b_off = blob_reserve(g, (size_t)L.n1pad * 4);
        L.w2_off = blob_reserve(g, (size_t)L.npad * K2 * 2);
        L.b2_off = blob_reserve(g, (size_t)L.npad * 4);
        uint16_t *w1 = reinterpret_cast<uint16_t *>(g.param_blob.data() + L.w_off);
        float *b1 = reinterpret_cast<float *>(g.param_blob.data() + L.b_off);
        uint16_t *w2 = reinterpret_cast<uint16_t *>(g.param_blob.data() + L.w2_off);
        float *b2 = reinterpret_cast<float *>(g.param_blob.data() + L.b2_off);
        for (int o = 0; o < A.cout; ++o) {
            for (int c = 0; c < src.c; ++c)
                for (int r = 0; r < A.k; ++r)
                    for (int s2 = 0; s2 < A.k; ++s2)
                        w1[(size_t)o * K1 + (r * A.k + s2) * src.c + c] = f32_to_bf16_rne(A.w[(((size_t)o * src.c + c) * A.k + r) * A.k + s2]);
            b1[o] = A.b[o];
        }
        auto pack2 = [&](const Node &n, int row0) {
            const int shift = (k2 - n.k) / 2;
            for (int o = 0; o < n.cout; ++o) {
                for (int c = 0; c < A.cout; ++c)
                    for (int r = 0; r < n.k; ++r)
                        for (int s2 = 0; s2 < n.k; ++s2)
                            w2[(size_t)(row0 + o) * K2 + ((r + shift) * k2 + (s2 + shift)) * L.n1pad + c] =
                                f32_to_bf16_rne(n.w[(((size_t)o * A.cout + c) * n.k + r) * n.k + s2]);
                b2[row0 + o] = n.b[o];
            }
        };
        if (B) pack2(*B, 0);
        else { pack2(*E0, 0); pack2(*E1, E0->cout); }
        for (int ni : cover) L.flops += 2.0 * node_macs(g.nodes[ni]);
        L.bytes = tbytes(L.in0) + tbytes(L.out) + (double)L.n1pad * K1 * 2 + (double)L.npad * K2 * 2 + 4.0 * (L.n1pad + L.npad);
        if (L.skip >= 0) L.bytes += tbytes(L.skip);
        push(L, ci);
        return XENOS_OK;
    }

    xenos_status_t lower_bf16_single(int ci, int ni) {
        const Node &n = g.nodes[ni];
        if (n.kind == NK_CONV) {
            // the first layer at small batch: a 3x3 convolution of an NCHW image runs on the CUDA cores (K = 27 fills
            // less than half of one 64-wide K block of the MMA; a launch of the persistent kernel costs more than this
            // whole layer).  Same-box A/B on MobileNet: batch 1 0.1506 -> 0.1424 ms; at batch 32 the tensor-core stem
            // with its TMA-fetched patches is faster (30 against 35.5 us), so larger batches keep it.
            const Tensor &x = g.tensors[n.in[0]];
            const bool no_request = !g.chains[ci].split.user;
            if (x.input_slot >= 0 && x.io_layout == XENOS_LAYOUT_NCHW && x.c <= 4 && n.k == 3 && (n.stride == 1 || n.stride == 2) &&
                n.cout % 8 == 0 && n.cout <= 64 && n.cin == x.c && no_request && !n.from_matmul && g.max_batch <= 8) {
                Launch L;
                L.kind = LK_STEM3X3;
                L.nodes = {ni};
                fill_io(L, n);
                L.seg[0].src_dtype = x.io_dtype;
                // weights [tap row][tap column][channel][cout], fp32
                std::vector<float> wt((size_t)9 * n.cin * n.cout);
                for (int o = 0; o < n.cout; ++o)
                    for (int c = 0; c < n.cin; ++c)
                        for (int t9 = 0; t9 < 9; ++t9) wt[((size_t)t9 * n.cin + c) * n.cout + o] = n.w[((size_t)o * n.cin + c) * 9 + t9];
                L.w_off = put_f32(wt); L.b_off = put_f32(n.b);
                L.flops = 2.0 * node_macs(n);
                L.bytes = tbytes(n.in[0]) + tbytes(n.out) + node_param_bytes(n);
                const int ih = 7 * n.stride + 3, iw = 31 * n.stride + 3;
                L.smem_bytes = 4 * (((n.cin * ih * (iw | 1) + 3) & ~3) + 9 * n.cin * n.cout + n.cout);
                L.grid = ceil_div(L.P, 8) * ceil_div(L.Q, 32);      // per image
                L.block = 256;
                push(L, ci);
                return XENOS_OK;
            }
        }
        if (n.kind == NK_CONV) return make_gemm(ci, {ni}, nullptr, &n, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, false);
        if (n.kind == NK_FC) {
            if (n.cin % 8) return fail(g, XENOS_E_UNSUPPORTED, "fc input length must be a multiple of 8");
            return make_gemm(ci, {ni}, nullptr, &n, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, true);
        }
        if (g.chains[ci].split.user && (g.chains[ci].split.outc > 1 || g.chains[ci].split.h > 1 || g.chains[ci].split.w > 1 || g.chains[ci].split.k > 1))
            return fail(g, XENOS_E_BAD_SPLIT, "split: element-wise, pooling and depthwise kernels are split one vector per thread; no explicit split");
        const Tensor &x = g.tensors[n.in[0]];
        if (!x.is_vec && x.c % 8) return fail(g, XENOS_E_UNSUPPORTED, "bf16 NHWC tensors need a channel count that is a multiple of 8");
        if (n.kind == NK_DW) {
            if (n.k != 3) return fail(g, XENOS_E_UNSUPPORTED, "depthwise convolution: only 3x3 has a kernel");
            Launch L;
            L.kind = LK_DW;
            L.nodes = {ni};
            fill_io(L, n);
            L.groups = n.cin;
            std::vector<float> wt((size_t)9 * n.cin);
            for (int c = 0; c < n.cin; ++c)
                for (int t = 0; t < 9; ++t) wt[(size_t)t * n.cin + c] = n.w[(size_t)c * 9 + t];
            L.w_off = put_f32(wt); L.b_off = put_f32(n.b);
            L.flops = 2.0 * node_macs(n);
            L.bytes = tbytes(n.in[0]) + tbytes(n.out) + node_param_bytes(n);
            L.block = 256;
            push(L, ci);
            return XENOS_OK;
        }
        return lower_single_common(ci, ni, false);
    }

    xenos_status_t lower_chain(int ci) {
        Chain &ch = g.chains[ci];
        // modelled traffic if every member ran alone (the unlinked baseline of the same chain)
        for (int ni : ch.nodes) {
            const Node &n = g.nodes[ni];
            ch.bytes_unlinked += tbytes(n.out) + node_param_bytes(n);
            for (int t : n.in) ch.bytes_unlinked += tbytes(t);
            ch.flops += 2.0 * node_macs(n);
        }
        xenos_status_t st = XENOS_OK;
        bool f32 = g.precision == XENOS_PRECISION_FP32_CUDA_CORE;
        auto find = [&](int kind, int nth = 0) -> const Node * {
            for (int ni : ch.nodes)
                if (g.nodes[ni].kind == kind && nth-- == 0) return &g.nodes[ni];
            return nullptr;
        };
        switch (ch.kind) {
        case CK_SINGLE:
            st = f32 ? lower_f32_single(ci, ch.nodes[0]) : lower_bf16_single(ci, ch.nodes[0]);
            break;
        case CK_CONV_CONV_POOL:
            st = lower_f32_linked(ci);
            break;
        case CK_DW_PW:
            st = make_gemm(ci, ch.nodes, find(NK_DW), find(NK_CONV), nullptr, nullptr, nullptr, nullptr, find(NK_GAP), nullptr, false);
            break;
        case CK_CONV_TAIL: {
            const Node *addn = find(NK_ADD);
            const Node *mainc = &g.nodes[ch.nodes[0]];
            const Node *sc = (addn && find(NK_CONV, 1)) ? find(NK_CONV, 1) : nullptr;
            st = make_gemm(ci, ch.nodes, nullptr, mainc, sc, nullptr, addn, find(NK_MAXPOOL), find(NK_GAP), nullptr, false);
            break;
        }
        case CK_MATMUL_MATMUL: {
            const Node &A = g.nodes[ch.nodes[0]], &B = g.nodes[ch.nodes[1]];
            Node M;                      // the one product that stands for both
            M.kind = A.kind; M.in = A.in; M.out = B.out; M.cin = A.cin; M.cout = B.cout; M.k = 1; M.stride = 1; M.pad = 0; M.act = B.act;
            M.w.assign((size_t)B.cout * A.cin, 0.0f);
            M.b.assign(B.cout, 0.0f);
            for (int o = 0; o < B.cout; ++o) {
                std::vector<double> row(A.cin, 0.0);
                double bias = B.b[o];
                for (int m = 0; m < A.cout; ++m) {
                    const double w2 = B.w[(size_t)o * A.cout + m];
                    bias += w2 * A.b[m];
                    const float *w1 = &A.w[(size_t)m * A.cin];
                    for (int c = 0; c < A.cin; ++c) row[c] += w2 * w1[c];
                }
                for (int c = 0; c < A.cin; ++c) M.w[(size_t)o * A.cin + c] = (float)row[c];
                M.b[o] = (float)bias;
            }
            st = make_gemm(ci, ch.nodes, nullptr, &M, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, A.kind == NK_FC);
            // (the modelled work of the launch is the merged product's, not the sum of the two it replaces)
            if (st == XENOS_OK) g.launches.back().flops = 2.0 * node_macs(M);
            break;
        }
        case CK_CONV_CONV: {
            const Node *cat = find(NK_CONCAT);
            if (cat) {
                const Node *first = &g.nodes[g.node_of_tensor[cat->in[0]]];
                const Node *second = &g.nodes[g.node_of_tensor[cat->in[1]]];
                st = make_gemm2(ci, ch.nodes, g.nodes[ch.nodes[0]], nullptr, first, second, nullptr, cat);
            } else {
                const Node *addn = find(NK_ADD);
                const Node &B = g.nodes[ch.nodes[1]];
                st = make_gemm2(ci, ch.nodes, g.nodes[ch.nodes[0]], &B, nullptr, nullptr, addn, addn ? addn : &B);
            }
            break;
        }
        case CK_EXPAND_CONCAT: {
            const Node *cat = find(NK_CONCAT);
            const Node *first = &g.nodes[g.node_of_tensor[cat->in[0]]];
            const Node *second = &g.nodes[g.node_of_tensor[cat->in[1]]];
            st = make_gemm(ci, ch.nodes, nullptr, first, nullptr, second, nullptr, find(NK_MAXPOOL), nullptr, cat, false);
            break;
        }
        default:
            st = fail(g, XENOS_E_UNSUPPORTED, "internal: unknown chain kind");
        }
        if (st != XENOS_OK) return st;
        for (int li : ch.launches) ch.bytes_linked += g.launches[li].bytes;
        return XENOS_OK;
    }
};

xenos_status_t split_and_lower(Graph &g) {
    g.launches.clear();
    g.param_blob.clear();
    Lower lw(g);
    for (int ci = 0; ci < (int)g.chains.size(); ++ci) {
        xenos_status_t st = lw.lower_chain(ci);
        if (st != XENOS_OK) return st;
    }
    return XENOS_OK;
}

// ------------------------------------------------------------------------------------------------
// Workspace: parameters, status words, then an arena for the tensors that live between kernels,
// placed first-fit by live interval (the memory-management part of the paper's runtime layer, Section 6).
// ------------------------------------------------------------------------------------------------
xenos_status_t plan_workspace(Graph &g) {
    int nt = (int)g.tensors.size();
    g.place.assign(nt, TensorPlace());
    bool f32 = g.precision == XENOS_PRECISION_FP32_CUDA_CORE;
    auto touch = [&](int t, int li, bool def) {
        if (t < 0) return;
        TensorPlace &p = g.place[t];
        p.materialised = true;
        if (p.first < 0 || (def && li < p.first)) p.first = p.first < 0 ? li : std::min(p.first, li);
        p.last = std::max(p.last, li);
    };
    for (int li = 0; li < (int)g.launches.size(); ++li) {
        const Launch &L = g.launches[li];
        touch(L.out, li, true);
        touch(L.in0, li, false); touch(L.in1, li, false); touch(L.in2, li, false); touch(L.skip, li, false);
        touch(L.seg[0].tensor, li, false); touch(L.seg[1].tensor, li, false);
    }
    size_t off = align_up(g.param_blob.size(), 256);
    g.status_off = off;
    off += 256;
    // arrival counters of the reduction-split launches sit behind the status words and are cleared with them
    g.cnt_bytes = 0; g.split_bytes = 0;
    for (Launch &L : g.launches)
        if (L.kind == LK_GEMM && L.ksplit > 1) {
            L.split_cnt_off = off + g.cnt_bytes;
            g.cnt_bytes += align_up((size_t)L.m_tiles * L.n_tiles * 8, 16);      // [arrived, reduced] per tile
            g.split_bytes = std::max(g.split_bytes, (size_t)L.ksplit * g.max_batch * L.rows_per_image * L.npad * 4);
        } else if (L.kind == LK_GEMM && L.gap_parts > 1) {
            L.split_cnt_off = off + g.cnt_bytes;
            g.cnt_bytes += align_up((size_t)g.max_batch * L.n_tiles * 8, 16);   // one counter per (image, channel tile)
            g.split_bytes = std::max(g.split_bytes, (size_t)g.max_batch * L.gap_parts * L.npad * 4);
        }
    g.cnt_bytes = align_up(g.cnt_bytes, 256);
    off += g.cnt_bytes;
    g.act_off = off;
    struct Live { size_t off, bytes; int last; };
    std::vector<Live> live;
    std::vector<int> order;
    for (int t = 0; t < nt; ++t) if (g.place[t].materialised) order.push_back(t);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return g.place[a].first < g.place[b].first; });
    size_t arena = 0;
    for (int t : order) {
        TensorPlace &p = g.place[t];
        const Tensor &x = g.tensors[t];
        if (f32) { p.dtype = XENOS_DTYPE_F32; p.layout = XENOS_LAYOUT_NCHW; }
        else { p.dtype = XENOS_DTYPE_BF16; p.layout = XENOS_LAYOUT_NHWC; }
        if (x.input_slot >= 0 || x.output_slot >= 0) {
            p.external = true;
            p.dtype = x.io_dtype; p.layout = x.io_layout;
            if (x.input_slot >= 0) p.first = 0;
            continue;
        }
        p.bytes = align_up((size_t)g.max_batch * tensor_elems(x) * (p.dtype == XENOS_DTYPE_F32 ? 4 : 2), 256);
        // lowest offset that overlaps no tensor still live when this one is defined
        std::vector<std::pair<size_t, size_t>> busy;
        for (const Live &l : live) if (l.last >= p.first) busy.push_back({l.off, l.off + l.bytes});
        std::sort(busy.begin(), busy.end());
        size_t cand = 0;
        for (auto &b : busy) {
            if (cand + p.bytes <= b.first) break;
            cand = std::max(cand, b.second);
        }
        p.off = g.act_off + cand;
        live.push_back({cand, p.bytes, p.last});
        arena = std::max(arena, cand + p.bytes);
    }
    g.split_off = align_up(g.act_off + arena, 256);
    g.workspace_bytes = g.split_off + g.split_bytes;
    // a graph input that is also read late must outlive everything: external, nothing to do.
    return XENOS_OK;
}

// ------------------------------------------------------------------------------------------------
// Plan as JSON
// ------------------------------------------------------------------------------------------------
static void jstr(std::string &s, const char *k, const std::string &v, bool comma = true) {
    s += "\""; s += k; s += "\":\""; s += v; s += "\""; if (comma) s += ",";
}
static void jint(std::string &s, const char *k, long long v, bool comma = true) {
    s += "\""; s += k; s += "\":"; s += std::to_string(v); if (comma) s += ",";
}
static void jdbl(std::string &s, const char *k, double v, bool comma = true) {
    char buf[64];
    snprintf(buf, sizeof buf, "%.0f", v);
    s += "\""; s += k; s += "\":"; s += buf; if (comma) s += ",";
}
static void jarr(std::string &s, const char *k, const std::vector<int> &v, bool comma = true) {
    s += "\""; s += k; s += "\":[";
    for (size_t i = 0; i < v.size(); ++i) { if (i) s += ","; s += std::to_string(v[i]); }
    s += "]"; if (comma) s += ",";
}

void emit_plan_json(Graph &g) {
    static const char *nk[] = {"?", "conv", "dwconv", "fc", "maxpool", "avgpool", "gap", "add", "concat", "mul", "mac", "transpose", "split"};
    static const char *ck[] = {"single", "conv_conv_pool", "dw_pw", "conv_tail", "expand_concat", "matmul_matmul", "conv_conv"};
    static const char *lk[] = {"?", "gemm", "dw", "pool", "gap", "add", "concat_part", "mulmac", "transpose", "slice", "f32_conv", "f32_pool",
                               "f32_gap", "f32_add", "f32_concat_part", "f32_fc", "f32_conv_conv_pool", "f32_mulmac", "f32_transpose", "f32_slice", "gemm2", "stem3x3"};
    static const char *am[] = {"none", "gather", "stem", "dw"};
    std::string s = "{";
    jstr(s, "precision", g.precision == XENOS_PRECISION_FP32_CUDA_CORE ? "fp32_cuda_core" : "bf16_tensor");
    jint(s, "max_batch", g.max_batch);
    s += "\"hw\":{";
    jint(s, "sm_count", g.hw.sm_count); jint(s, "smem_bytes_per_cta", g.hw.smem_bytes_per_cta);
    jint(s, "tmem_columns", g.hw.tmem_columns); jint(s, "l2_bytes", g.hw.l2_bytes, false);
    s += "},";
    jstr(s, "cta_to_tile", "gemm: cta = m_tile * n_tiles + n_tile, tiles dealt to units round-robin in ascending order; "
                            "f32 chain: cta = ((image * parts_outc + outc_part) * tiles_h + tile_y) * tiles_w + tile_x");
    s += "\"nodes\":[";
    for (size_t i = 0; i < g.nodes.size(); ++i) {
        const Node &n = g.nodes[i];
        if (i) s += ",";
        s += "{";
        jint(s, "id", (long long)i); jstr(s, "kind", nk[n.kind]); jarr(s, "in", n.in); jint(s, "out", n.out);
        jint(s, "cin", n.cin); jint(s, "cout", n.cout); jint(s, "k", n.k); jint(s, "stride", n.stride);
        jint(s, "pad", n.pad); jint(s, "act", n.act); jarr(s, "user_ops", n.user_ops); jint(s, "chain", n.chain, false);
        s += "}";
    }
    s += "],\"chains\":[";
    double tf = 0, tb = 0, tu = 0;
    for (size_t i = 0; i < g.chains.size(); ++i) {
        const Chain &c = g.chains[i];
        if (i) s += ",";
        s += "{";
        jint(s, "id", (long long)i); jstr(s, "kind", ck[c.kind]); jstr(s, "pattern", c.pattern);
        jarr(s, "nodes", c.nodes); jarr(s, "launches", c.launches);
        jdbl(s, "flops", c.flops); jdbl(s, "bytes_linked", c.bytes_linked); jdbl(s, "bytes_unlinked", c.bytes_unlinked, false);
        s += "}";
        tf += c.flops; tb += c.bytes_linked; tu += c.bytes_unlinked;
    }
    s += "],\"launches\":[";
    for (size_t i = 0; i < g.launches.size(); ++i) {
        const Launch &L = g.launches[i];
        if (i) s += ",";
        s += "{";
        jint(s, "id", (long long)i); jstr(s, "kind", lk[L.kind]); jint(s, "chain", L.chain); jarr(s, "nodes", L.nodes);
        jint(s, "in0", L.in0); jint(s, "in1", L.in1); jint(s, "in2", L.in2); jint(s, "skip", L.skip); jint(s, "out", L.out);
        jint(s, "out_coff", L.out_coff); jint(s, "out_ctot", L.out_ctot);
        jint(s, "C", L.C); jint(s, "H", L.H); jint(s, "W", L.W); jint(s, "K", L.K); jint(s, "P", L.P); jint(s, "Q", L.Q);
        jint(s, "k", L.k); jint(s, "stride", L.stride); jint(s, "pad", L.pad);
        if (L.kind == LK_GEMM) {
            jstr(s, "a0", am[L.seg[0].mode]); jstr(s, "a1", am[L.seg[1].mode]);
            jint(s, "kblocks", L.kblocks); jint(s, "npad", L.npad); jint(s, "tile_m", 128); jint(s, "tile_n", L.tile_n);
            jint(s, "tile_k", 64); jint(s, "n_tiles", L.n_tiles); jint(s, "m_tiles", L.m_tiles);
            jint(s, "tile_rows", L.tile_rows); jint(s, "epi", L.epi); jint(s, "map", L.map_mode);
            jint(s, "imgs_per_tile", L.imgs_per_tile);
            jint(s, "patch_th", L.patch_th); jint(s, "patch_tw", L.patch_tw); jint(s, "patch_rh", L.patch_rh);
            jint(s, "patch_rw", L.patch_rw); jint(s, "tiles_y", L.tiles_y); jint(s, "tiles_x", L.tiles_x);
            jint(s, "stages", L.stages); jint(s, "tmem_cols", L.tmem_cols); jint(s, "acc_stride", L.acc_stride);
            jint(s, "ni", L.ni); jint(s, "step_y", L.step_y); jint(s, "step_x", L.step_x); jint(s, "off_y", L.off_y); jint(s, "off_x", L.off_x);
            jint(s, "hstages", L.hstages); jint(s, "halo_h", L.halo_h); jint(s, "halo_w", L.halo_w); jint(s, "halo_cb", L.halo_cb);
            jint(s, "halo_bytes", L.halo_bytes);
            jint(s, "ksplit", L.ksplit); jint(s, "kb_per", L.kb_per); jint(s, "a_tma", L.a_tma); jint(s, "fc_small", L.fc_small); jint(s, "dw_workers", L.dw_workers); jint(s, "n_acc", L.n_acc); jint(s, "gap_parts", L.gap_parts);
        }
        if (L.kind == LK_GEMM2) {
            jint(s, "k2", L.k2); jint(s, "cmid", L.Cmid); jint(s, "n1pad", L.n1pad); jint(s, "kblocks", L.kblocks); jint(s, "kblocks2", L.kblocks2);
            jint(s, "tile_n", L.tile_n); jint(s, "n_tiles", L.n_tiles); jint(s, "m_tiles", L.m_tiles); jint(s, "npad", L.npad);
            jint(s, "patch_rh", L.patch_rh); jint(s, "patch_rw", L.patch_rw); jint(s, "rh2", L.rh2); jint(s, "rw2", L.rw2);
            jint(s, "tiles_y", L.tiles_y); jint(s, "tiles_x", L.tiles_x); jint(s, "stages", L.stages);
        }
        if (L.kind == LK_F32_CONV_CONV_POOL) {
            jint(s, "parts_outc", L.parts_outc); jint(s, "tile_h", L.tile_h); jint(s, "tile_w", L.tile_w);
            jint(s, "tiles_h", L.tiles_h); jint(s, "tiles_w", L.tiles_w); jint(s, "halo_h", L.halo_h); jint(s, "halo_w", L.halo_w);
        }
        jint(s, "w_off", (long long)L.w_off); jint(s, "b_off", (long long)L.b_off);
        jint(s, "smem_bytes", L.smem_bytes); jint(s, "grid", L.grid); jint(s, "block", L.block);
        jdbl(s, "flops", L.flops); jdbl(s, "bytes", L.bytes, false);
        s += "}";
    }
    s += "],\"tensors\":[";
    bool firstt = true;
    for (size_t t = 0; t < g.tensors.size(); ++t) {
        const TensorPlace &p = g.place[t];
        if (!p.materialised) continue;
        if (!firstt) s += ",";
        firstt = false;
        const Tensor &x = g.tensors[t];
        s += "{";
        jint(s, "id", (long long)t); jint(s, "c", x.c); jint(s, "h", x.h); jint(s, "w", x.w);
        jint(s, "external", p.external); jint(s, "off", (long long)p.off); jint(s, "bytes", (long long)p.bytes);
        jint(s, "first", p.first); jint(s, "last", p.last, false);
        s += "}";
    }
    s += "],";
    jint(s, "param_bytes", (long long)g.param_blob.size());
    jint(s, "workspace_bytes", (long long)g.workspace_bytes);
    jdbl(s, "flops", tf); jdbl(s, "bytes_linked", tb); jdbl(s, "bytes_unlinked", tu, false);
    s += "}";
    g.plan_json.swap(s);
}

}  // namespace xenos
