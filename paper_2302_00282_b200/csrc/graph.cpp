// Graph construction with shape inference, and the compile driver.
#include "graph.hpp"

#include <cmath>

namespace xenos {

static bool finite_all(const float *p, size_t n) {
    for (size_t i = 0; i < n; ++i)
        if (!std::isfinite(p[i])) return false;
    return true;
}

// Appends one user operator; the output extent of window operators is
// floor((in + 2*pad - k) / stride) + 1.
xenos_status_t infer_and_append(Graph &g, const xenos_op_desc_t &d, const int *in, int n_in, int *out) {
    for (int i = 0; i < n_in; ++i)
        if (in[i] < 0 || in[i] >= (int)g.tensors.size()) return fail(g, XENOS_E_INVALID, "add_op: bad input tensor id");
    const Tensor x = g.tensors[in[0]];
    Op op;
    op.kind = d.kind;
    op.in.assign(in, in + n_in);
    Tensor y;
    auto need_inputs = [&](int n) { return n_in == n; };
    bool has_bn = d.bn_gamma || d.bn_beta || d.bn_mean || d.bn_var;
    if (has_bn && !(d.bn_gamma && d.bn_beta && d.bn_mean && d.bn_var))
        return fail(g, XENOS_E_INVALID, "add_op: BatchNorm needs gamma, beta, mean and var together");
    if (d.act != XENOS_ACT_NONE && d.act != XENOS_ACT_RELU && d.act != XENOS_ACT_RELU6)
        return fail(g, XENOS_E_INVALID, "add_op: unknown activation");

    switch (d.kind) {
    case XENOS_OP_CONV: {
        if (!need_inputs(1)) return fail(g, XENOS_E_INVALID, "conv takes one input");
        if (x.is_vec) return fail(g, XENOS_E_SHAPE, "conv input must be a feature map");
        if (!d.weight) return fail(g, XENOS_E_INVALID, "conv: weight is NULL");
        if (d.kh != d.kw) return fail(g, XENOS_E_UNSUPPORTED, "conv: only square kernels");
        if (d.kh < 1 || d.stride < 1 || d.pad < 0 || d.cout < 1 || d.groups < 1)
            return fail(g, XENOS_E_SHAPE, "conv: bad kernel / stride / pad / cout / groups");
        if (x.c % d.groups || d.cout % d.groups) return fail(g, XENOS_E_SHAPE, "conv: groups must divide Cin and Cout");
        if (d.groups != 1 && !(d.groups == x.c && d.cout == x.c))
            return fail(g, XENOS_E_UNSUPPORTED, "conv: groups must be 1 (dense) or Cin == Cout (depthwise)");
        y.c = d.cout;
        y.h = out_dim(x.h, d.kh, d.stride, d.pad);
        y.w = out_dim(x.w, d.kh, d.stride, d.pad);
        if (y.h < 1 || y.w < 1) return fail(g, XENOS_E_SHAPE, "conv: kernel larger than padded input");
        size_t nw = (size_t)d.cout * (x.c / d.groups) * d.kh * d.kh;
        if (!finite_all(d.weight, nw)) return fail(g, XENOS_E_INVALID, "conv: non-finite weight");
        op.w.assign(d.weight, d.weight + nw);
        op.cout = d.cout; op.k = d.kh; op.stride = d.stride; op.pad = d.pad; op.groups = d.groups;
        break;
    }
    case XENOS_OP_FC: {
        if (!need_inputs(1)) return fail(g, XENOS_E_INVALID, "fc takes one input");
        if (!x.is_vec) return fail(g, XENOS_E_SHAPE, "fc input must be a vector (e.g. a global pool output)");
        if (!d.weight || d.cout < 1) return fail(g, XENOS_E_INVALID, "fc: weight is NULL or cout < 1");
        size_t nw = (size_t)d.cout * x.c;
        if (!finite_all(d.weight, nw)) return fail(g, XENOS_E_INVALID, "fc: non-finite weight");
        op.w.assign(d.weight, d.weight + nw);
        op.cout = d.cout; op.k = 1; op.groups = 1;
        y.c = d.cout; y.is_vec = true;
        break;
    }
    case XENOS_OP_POOL_MAX:
    case XENOS_OP_POOL_AVG: {
        if (!need_inputs(1)) return fail(g, XENOS_E_INVALID, "pool takes one input");
        if (x.is_vec) return fail(g, XENOS_E_SHAPE, "pool input must be a feature map");
        if (d.kh != d.kw || d.kh < 1 || d.stride < 1 || d.pad < 0) return fail(g, XENOS_E_SHAPE, "pool: bad window");
        if (d.pad >= d.kh) return fail(g, XENOS_E_SHAPE, "pool: pad must be smaller than the window");
        if (d.kind == XENOS_OP_POOL_AVG && d.pad != 0)
            return fail(g, XENOS_E_UNSUPPORTED, "avg pool with padding is not implemented");
        y.c = x.c;
        y.h = out_dim(x.h, d.kh, d.stride, d.pad);
        y.w = out_dim(x.w, d.kh, d.stride, d.pad);
        if (y.h < 1 || y.w < 1) return fail(g, XENOS_E_SHAPE, "pool: window larger than padded input");
        op.k = d.kh; op.stride = d.stride; op.pad = d.pad;
        break;
    }
    case XENOS_OP_POOL_GLOBAL_AVG:
        if (!need_inputs(1)) return fail(g, XENOS_E_INVALID, "global pool takes one input");
        if (x.is_vec) return fail(g, XENOS_E_SHAPE, "global pool input must be a feature map");
        y.c = x.c; y.is_vec = true;
        break;
    case XENOS_OP_ADD: {
        if (!need_inputs(2)) return fail(g, XENOS_E_INVALID, "add takes two inputs");
        const Tensor &b = g.tensors[in[1]];
        if (x.c != b.c || x.h != b.h || x.w != b.w || x.is_vec != b.is_vec)
            return fail(g, XENOS_E_SHAPE, "add: operand shapes differ");
        y.c = x.c; y.h = x.h; y.w = x.w; y.is_vec = x.is_vec;
        break;
    }
    case XENOS_OP_CONCAT: {
        if (n_in < 2) return fail(g, XENOS_E_INVALID, "concat takes at least two inputs");
        if (x.is_vec) return fail(g, XENOS_E_SHAPE, "concat inputs must be feature maps");
        int c = 0;
        for (int i = 0; i < n_in; ++i) {
            const Tensor &t = g.tensors[in[i]];
            if (t.is_vec || t.h != x.h || t.w != x.w) return fail(g, XENOS_E_SHAPE, "concat: spatial extents differ");
            c += t.c;
        }
        y.c = c; y.h = x.h; y.w = x.w;
        break;
    }
    case XENOS_OP_RELU:
    case XENOS_OP_RELU6:
        if (!need_inputs(1)) return fail(g, XENOS_E_INVALID, "activation takes one input");
        y.c = x.c; y.h = x.h; y.w = x.w; y.is_vec = x.is_vec;
        break;
    case XENOS_OP_BATCHNORM:
        if (!need_inputs(1)) return fail(g, XENOS_E_INVALID, "batchnorm takes one input");
        if (!has_bn) return fail(g, XENOS_E_INVALID, "batchnorm: parameters are NULL");
        y.c = x.c; y.h = x.h; y.w = x.w; y.is_vec = x.is_vec;
        break;
    case XENOS_OP_MUL:
    case XENOS_OP_MAC: {
        const int need = d.kind == XENOS_OP_MUL ? 2 : 3;
        if (!need_inputs(need)) return fail(g, XENOS_E_INVALID, d.kind == XENOS_OP_MUL ? "mul takes two inputs" : "mac takes three inputs");
        for (int i = 1; i < need; ++i) {
            const Tensor &b = g.tensors[in[i]];
            if (x.c != b.c || x.h != b.h || x.w != b.w || x.is_vec != b.is_vec)
                return fail(g, XENOS_E_SHAPE, "mul / mac: operand shapes differ");
        }
        y.c = x.c; y.h = x.h; y.w = x.w; y.is_vec = x.is_vec;
        break;
    }
    case XENOS_OP_TRANSPOSE:
        if (!need_inputs(1)) return fail(g, XENOS_E_INVALID, "transpose takes one input");
        if (x.is_vec || x.w != 1) return fail(g, XENOS_E_SHAPE, "transpose input must be a matrix (a feature map of width 1)");
        y.c = x.h; y.h = x.c; y.w = 1;
        break;
    case XENOS_OP_SPLIT:
        if (!need_inputs(1)) return fail(g, XENOS_E_INVALID, "split takes one input");
        if (x.is_vec) return fail(g, XENOS_E_SHAPE, "split input must be a feature map");
        if (d.cout < 1 || d.pad < 0 || d.pad + d.cout > x.c) return fail(g, XENOS_E_SHAPE, "split: channels [pad, pad + cout) leave the input");
        y.c = d.cout; y.h = x.h; y.w = x.w;
        op.cout = d.cout; op.pad = d.pad;
        break;
    case XENOS_OP_MATMUL: {
        if (n_in == 2) return fail(g, XENOS_E_UNSUPPORTED, "matmul of two run-time tensors is not implemented; the right operand is a constant (weight)");
        if (!need_inputs(1)) return fail(g, XENOS_E_INVALID, "matmul takes one input and a constant matrix");
        if (!x.is_vec && x.w != 1) return fail(g, XENOS_E_SHAPE, "matmul input must be a matrix (a feature map of width 1) or a vector");
        if (!d.weight || d.cout < 1) return fail(g, XENOS_E_INVALID, "matmul: weight is NULL or cout < 1");
        size_t nw = (size_t)x.c * d.cout;
        if (!finite_all(d.weight, nw)) return fail(g, XENOS_E_INVALID, "matmul: non-finite weight");
        // kept as [cout][c], the form of a pointwise convolution / fc
        op.w.resize(nw);
        for (int k = 0; k < x.c; ++k)
            for (int n = 0; n < d.cout; ++n) op.w[(size_t)n * x.c + k] = d.weight[(size_t)k * d.cout + n];
        op.cout = d.cout; op.k = 1; op.groups = 1;
        y.c = d.cout; y.h = x.h; y.w = x.w; y.is_vec = x.is_vec;
        break;
    }
    default:
        return fail(g, XENOS_E_UNSUPPORTED, "add_op: unknown operator kind");
    }

    int cpar = (d.kind == XENOS_OP_BATCHNORM) ? x.c : d.cout;
    if (d.kind == XENOS_OP_CONV || d.kind == XENOS_OP_FC || d.kind == XENOS_OP_MATMUL) {
        op.act = d.act;
        if (d.bias) {
            if (!finite_all(d.bias, d.cout)) return fail(g, XENOS_E_INVALID, "non-finite bias");
            op.bias.assign(d.bias, d.bias + d.cout);
            op.has_bias = true;
        }
    } else if (d.act != XENOS_ACT_NONE && d.kind != XENOS_OP_ADD) {
        return fail(g, XENOS_E_INVALID, "add_op: activation only attaches to conv, fc and add");
    } else {
        op.act = d.act;
    }
    if (has_bn) {
        if (d.kind != XENOS_OP_CONV && d.kind != XENOS_OP_FC && d.kind != XENOS_OP_MATMUL && d.kind != XENOS_OP_BATCHNORM)
            return fail(g, XENOS_E_INVALID, "add_op: BatchNorm parameters on an operator that cannot carry them");
        if (!(d.bn_eps > 0.0f)) return fail(g, XENOS_E_INVALID, "batchnorm: eps must be positive");
        if (!finite_all(d.bn_gamma, cpar) || !finite_all(d.bn_beta, cpar) || !finite_all(d.bn_mean, cpar) ||
            !finite_all(d.bn_var, cpar))
            return fail(g, XENOS_E_INVALID, "batchnorm: non-finite parameter");
        for (int i = 0; i < cpar; ++i)
            if (!(d.bn_var[i] + d.bn_eps > 0.0f)) return fail(g, XENOS_E_INVALID, "batchnorm: var + eps must be positive");
        op.gamma.assign(d.bn_gamma, d.bn_gamma + cpar);
        op.beta.assign(d.bn_beta, d.bn_beta + cpar);
        op.mean.assign(d.bn_mean, d.bn_mean + cpar);
        op.var.assign(d.bn_var, d.bn_var + cpar);
        op.eps = d.bn_eps;
        op.has_bn = true;
    }

    int opi = (int)g.ops.size();
    y.producer = opi;
    g.tensors.push_back(y);
    op.out = (int)g.tensors.size() - 1;
    for (int i = 0; i < n_in; ++i) g.tensors[in[i]].consumers.push_back(opi);
    g.ops.push_back(std::move(op));
    *out = g.ops.back().out;
    return XENOS_OK;
}

xenos_status_t compile_graph(Graph &g, int max_batch, int precision) {
    if (g.inputs.empty()) return fail(g, XENOS_E_INVALID, "compile: graph has no input");
    if (g.outputs.empty()) return fail(g, XENOS_E_INVALID, "compile: graph has no output");
    if (g.ops.empty()) return fail(g, XENOS_E_INVALID, "compile: graph has no operator");
    g.precision = precision;
    g.max_batch = max_batch;
    for (int t : g.inputs) {
        const Tensor &x = g.tensors[t];
        if (precision == XENOS_PRECISION_FP32_CUDA_CORE &&
            (x.io_dtype != XENOS_DTYPE_F32 || x.io_layout != XENOS_LAYOUT_NCHW))
            return fail(g, XENOS_E_UNSUPPORTED, "fp32 graphs take F32 NCHW inputs");
    }
    for (int t : g.outputs) {
        const Tensor &x = g.tensors[t];
        if (precision == XENOS_PRECISION_FP32_CUDA_CORE) {
            if (x.io_dtype != XENOS_DTYPE_F32 || (!x.is_vec && x.io_layout != XENOS_LAYOUT_NCHW))
                return fail(g, XENOS_E_UNSUPPORTED, "fp32 graphs produce F32 NCHW outputs");
        } else {
            if (x.is_vec && x.io_dtype != XENOS_DTYPE_F32)
                return fail(g, XENOS_E_UNSUPPORTED, "bf16 graphs produce vector outputs in F32");
            if (!x.is_vec && (x.io_dtype != XENOS_DTYPE_BF16 || x.io_layout != XENOS_LAYOUT_NHWC))
                return fail(g, XENOS_E_UNSUPPORTED, "bf16 graphs produce feature-map outputs as BF16 NHWC");
        }
    }
    xenos_status_t st;
    if ((st = prefuse(g)) != XENOS_OK) return st;
    if ((st = link_pass(g)) != XENOS_OK) return st;
    if ((st = split_and_lower(g)) != XENOS_OK) return st;
    if ((st = plan_workspace(g)) != XENOS_OK) return st;
    emit_plan_json(g);
    return XENOS_OK;
}

}  // namespace xenos
