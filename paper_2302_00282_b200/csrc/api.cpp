// C ABI of the library: argument checks, the call-order state machine, and dispatch into the
// host passes and the CUDA runtime.  No exception leaves this file.
#include <atomic>
#include <cstring>
#include <new>
#include <string>

#include "graph.hpp"

using namespace xenos;

struct xenos_graph {
    Graph g;
};

namespace xenos {
xenos_status_t fail(const Graph &g, xenos_status_t code, const std::string &msg) {
    g.err = msg;
    return code;
}
}  // namespace xenos

static thread_local std::string g_create_err;

#define XENOS_GUARD_BEGIN try {
#define XENOS_GUARD_END(gptr)                                                         \
    }                                                                                 \
    catch (const std::bad_alloc &) {                                                  \
        if (gptr) (gptr)->g.err = "out of host memory";                               \
        return XENOS_E_INVALID;                                                       \
    }                                                                                 \
    catch (const std::exception &e) {                                                 \
        if (gptr) (gptr)->g.err = std::string("internal error: ") + e.what();         \
        return XENOS_E_INVALID;                                                       \
    }                                                                                 \
    catch (...) {                                                                     \
        if (gptr) (gptr)->g.err = "internal error";                                   \
        return XENOS_E_INVALID;                                                       \
    }

// Shared argument checks of the three run entry points.  Device buffers are read and written with
// 16-byte vector accesses and by TMA, so every input and output pointer must be 16-byte aligned.
static xenos_status_t check_run_args(const Graph &g, const char *who, int32_t batch, const void *const *inputs_dev,
                                     void *const *outputs_dev) {
    const std::string w(who);
    if (batch < 1 || batch > g.max_batch) return fail(g, XENOS_E_INVALID, w + ": batch exceeds max_batch given to compile");
    if (!inputs_dev || !outputs_dev) return fail(g, XENOS_E_INVALID, w + ": NULL pointer array");
    for (size_t i = 0; i < g.inputs.size(); ++i) {
        if (!inputs_dev[i]) return fail(g, XENOS_E_INVALID, w + ": NULL input pointer");
        if ((uintptr_t)inputs_dev[i] & 15u) return fail(g, XENOS_E_INVALID, w + ": input pointer is not 16-byte aligned");
    }
    for (size_t i = 0; i < g.outputs.size(); ++i) {
        if (!outputs_dev[i]) return fail(g, XENOS_E_INVALID, w + ": NULL output pointer");
        if ((uintptr_t)outputs_dev[i] & 15u) return fail(g, XENOS_E_INVALID, w + ": output pointer is not 16-byte aligned");
    }
    return XENOS_OK;
}

extern "C" {

xenos_status_t xenos_graph_create(const xenos_hw_info_t *hw, xenos_graph_t **out) {
    if (!out) {
        g_create_err = "xenos_graph_create: out is NULL";
        return XENOS_E_INVALID;
    }
    *out = nullptr;
    xenos_graph *p = new (std::nothrow) xenos_graph();
    if (!p) {
        g_create_err = "out of host memory";
        return XENOS_E_INVALID;
    }
    if (hw) {
        if (hw->sm_count < 1 || hw->smem_bytes_per_cta < 48 * 1024 || hw->tmem_columns < 32 ||
            hw->tmem_columns > 512 || hw->l2_bytes < 0) {
            delete p;
            g_create_err = "xenos_graph_create: hardware info out of range";
            return XENOS_E_INVALID;
        }
        p->g.hw = *hw;
    }
    static std::atomic<uint64_t> next_serial{1};
    p->g.serial = next_serial.fetch_add(1);
    *out = p;
    return XENOS_OK;
}

xenos_status_t xenos_graph_add_input(xenos_graph_t *gp, int32_t dtype, int32_t layout, int32_t c,
                                     int32_t h, int32_t w, xenos_id_t *tensor) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state != ST_BUILD) return fail(g, XENOS_E_STATE, "add_input after compile");
    if (!tensor) return fail(g, XENOS_E_INVALID, "add_input: tensor is NULL");
    if ((dtype != XENOS_DTYPE_F32 && dtype != XENOS_DTYPE_BF16) ||
        (layout != XENOS_LAYOUT_NCHW && layout != XENOS_LAYOUT_NHWC))
        return fail(g, XENOS_E_INVALID, "add_input: unknown dtype or layout");
    if (c < 1 || h < 1 || w < 1) return fail(g, XENOS_E_SHAPE, "add_input: extents must be positive");
    Tensor t;
    t.c = c; t.h = h; t.w = w;
    t.input_slot = (int)g.inputs.size();
    t.io_dtype = dtype; t.io_layout = layout;
    g.tensors.push_back(t);
    g.inputs.push_back((int)g.tensors.size() - 1);
    *tensor = (int)g.tensors.size() - 1;
    return XENOS_OK;
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_add_op(xenos_graph_t *gp, const xenos_op_desc_t *desc, const xenos_id_t *inputs,
                                  int32_t n_inputs, xenos_id_t *out_tensor) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state != ST_BUILD) return fail(g, XENOS_E_STATE, "add_op after compile");
    if (!desc || !inputs || !out_tensor || n_inputs < 1)
        return fail(g, XENOS_E_INVALID, "add_op: NULL argument or no inputs");
    return infer_and_append(g, *desc, inputs, n_inputs, out_tensor);
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_mark_output(xenos_graph_t *gp, xenos_id_t tensor, int32_t dtype, int32_t layout) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state != ST_BUILD) return fail(g, XENOS_E_STATE, "mark_output after compile");
    if (tensor < 0 || tensor >= (int)g.tensors.size()) return fail(g, XENOS_E_INVALID, "mark_output: bad tensor id");
    if ((dtype != XENOS_DTYPE_F32 && dtype != XENOS_DTYPE_BF16) ||
        (layout != XENOS_LAYOUT_NCHW && layout != XENOS_LAYOUT_NHWC))
        return fail(g, XENOS_E_INVALID, "mark_output: unknown dtype or layout");
    Tensor &t = g.tensors[tensor];
    if (t.input_slot >= 0) return fail(g, XENOS_E_INVALID, "mark_output: a graph input cannot be an output");
    if (t.output_slot >= 0) return fail(g, XENOS_E_INVALID, "mark_output: tensor is already an output");
    t.output_slot = (int)g.outputs.size();
    t.io_dtype = dtype; t.io_layout = layout;
    g.outputs.push_back(tensor);
    return XENOS_OK;
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_link(xenos_graph_t *gp, const xenos_id_t *ops, int32_t n_ops) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state != ST_BUILD) return fail(g, XENOS_E_STATE, "link after compile");
    if (n_ops < 0 || (n_ops > 0 && !ops)) return fail(g, XENOS_E_INVALID, "link: bad arguments");
    if (n_ops == 0) {
        g.link_auto = true;
        return XENOS_OK;
    }
    if (n_ops < 2) return fail(g, XENOS_E_NOT_LINKABLE, "link: a chain needs at least two operators");
    LinkRequest r;
    for (int i = 0; i < n_ops; ++i) {
        if (ops[i] < 0 || ops[i] >= (int)g.tensors.size() || g.tensors[ops[i]].producer < 0)
            return fail(g, XENOS_E_INVALID, "link: id is not an operator output");
        r.ops.push_back(ops[i]);
    }
    // adjacency is checked here so that a bad request fails at the call that made it: every operator after the
    // first must read an earlier operator of the list (the one before it in a plain chain; the squeeze convolution
    // for both expands of a fire module), possibly through the bn / activation records that follow that operator
    for (int i = 0; i + 1 < n_ops; ++i) {
        const Op &nx = g.ops[g.tensors[r.ops[i + 1]].producer];
        bool found = false;
        for (int t : nx.in) {
            int cur = t;
            for (int hop = 0; hop < 3 && cur >= 0; ++hop) {
                for (int e = 0; e <= i; ++e) if (cur == r.ops[e]) found = true;
                if (found) break;
                int p = g.tensors[cur].producer;
                if (p < 0) break;
                int kd = g.ops[p].kind;
                if (kd != XENOS_OP_BATCHNORM && kd != XENOS_OP_RELU && kd != XENOS_OP_RELU6) break;
                cur = g.ops[p].in[0];
            }
            if (found) break;
        }
        if (!found) return fail(g, XENOS_E_NOT_LINKABLE, "link: operators are not adjacent producer -> consumer");
    }
    g.link_requests.push_back(r);
    return XENOS_OK;
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_split(xenos_graph_t *gp, xenos_id_t op, int32_t parts_outc, int32_t parts_h,
                                 int32_t parts_w, int32_t parts_k) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state != ST_BUILD) return fail(g, XENOS_E_STATE, "split after compile");
    if (op == -1) return XENOS_OK;   // automatic split is the default for every chain
    if (op < 0 || op >= (int)g.tensors.size() || g.tensors[op].producer < 0)
        return fail(g, XENOS_E_INVALID, "split: id is not an operator output");
    if (parts_outc < 0 || parts_h < 0 || parts_w < 0 || parts_k < 0)
        return fail(g, XENOS_E_BAD_SPLIT, "split: negative part count");
    SplitRequest s;
    s.outc = parts_outc; s.h = parts_h; s.w = parts_w; s.k = parts_k > 1 ? parts_k : 1; s.user = true;
    g.split_requests.push_back({op, s});
    return XENOS_OK;
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_search_split(xenos_graph_t *gp, int32_t max_batch, int32_t precision, void *workspace_dev,
                                        size_t workspace_bytes, const void *const *inputs_dev, void *const *outputs_dev,
                                        void *cuda_stream, int32_t max_trials, int32_t repeats, char *report_json, size_t cap,
                                        size_t *needed) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state != ST_BUILD) return fail(g, XENOS_E_STATE, "search_split after compile");
    if (max_batch < 1 || max_batch > 65535) return fail(g, XENOS_E_INVALID, "search_split: max_batch out of range");
    if (precision != XENOS_PRECISION_FP32_CUDA_CORE && precision != XENOS_PRECISION_BF16_TENSOR)
        return fail(g, XENOS_E_INVALID, "search_split: unknown precision");
    if (!workspace_dev || ((uintptr_t)workspace_dev & 255u)) return fail(g, XENOS_E_WORKSPACE, "search_split: workspace is NULL or not 256-byte aligned");
    if (max_trials < 1 || max_trials > 64 || repeats < 1 || repeats > 1000) return fail(g, XENOS_E_INVALID, "search_split: max_trials must be 1..64 and repeats 1..1000");
    if (!inputs_dev || !outputs_dev || !needed) return fail(g, XENOS_E_INVALID, "search_split: NULL pointer");
    for (size_t i = 0; i < g.inputs.size(); ++i)
        if (!inputs_dev[i] || ((uintptr_t)inputs_dev[i] & 15u)) return fail(g, XENOS_E_INVALID, "search_split: input pointer is NULL or not 16-byte aligned");
    for (size_t i = 0; i < g.outputs.size(); ++i)
        if (!outputs_dev[i] || ((uintptr_t)outputs_dev[i] & 15u)) return fail(g, XENOS_E_INVALID, "search_split: output pointer is NULL or not 16-byte aligned");
    std::string report;
    xenos_status_t st = search_splits(g, max_batch, precision, workspace_dev, workspace_bytes, inputs_dev, outputs_dev, cuda_stream,
                                      max_trials, repeats, report);
    if (st != XENOS_OK) return st;
    *needed = report.size() + 1;
    if (report_json && cap > 0) {
        size_t n = report.size() < cap - 1 ? report.size() : cap - 1;
        std::memcpy(report_json, report.data(), n);
        report_json[n] = '\0';
    }
    return XENOS_OK;
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_compile(xenos_graph_t *gp, int32_t max_batch, int32_t precision, size_t *workspace_bytes) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state != ST_BUILD) return fail(g, XENOS_E_STATE, "compile called twice");
    if (!workspace_bytes) return fail(g, XENOS_E_INVALID, "compile: workspace_bytes is NULL");
    if (max_batch < 1 || max_batch > 65535) return fail(g, XENOS_E_INVALID, "compile: max_batch out of range");
    if (precision != XENOS_PRECISION_FP32_CUDA_CORE && precision != XENOS_PRECISION_BF16_TENSOR)
        return fail(g, XENOS_E_INVALID, "compile: unknown precision");
    xenos_status_t st = compile_graph(g, max_batch, precision);
    if (st != XENOS_OK) {
        // leave the graph in build state, drop partial results
        g.nodes.clear(); g.chains.clear(); g.launches.clear(); g.place.clear(); g.param_blob.clear();
        g.node_of_tensor.clear(); g.plan_json.clear();
        return st;
    }
    g.state = ST_COMPILED;
    *workspace_bytes = g.workspace_bytes;
    return XENOS_OK;
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_save(const xenos_graph_t *gp, void *host_buf, size_t cap, size_t *needed) {
    if (!gp) return XENOS_E_INVALID;
    const Graph &g = gp->g;
    try {
        if (!needed) return fail(g, XENOS_E_INVALID, "save: needed is NULL");
        std::vector<uint8_t> img;
        save_graph(g, img);
        *needed = img.size();
        if (!host_buf) return XENOS_OK;              // size query
        if (cap < img.size()) return fail(g, XENOS_E_INVALID, "save: the buffer is smaller than the image");
        std::memcpy(host_buf, img.data(), img.size());
        return XENOS_OK;
    } catch (const std::exception &e) {
        return fail(g, XENOS_E_INVALID, std::string("save: ") + e.what());
    }
}

xenos_status_t xenos_graph_load(const void *host_buf, size_t bytes, xenos_graph_t **out, size_t *workspace_bytes) {
    if (!out) {
        g_create_err = "xenos_graph_load: out is NULL";
        return XENOS_E_INVALID;
    }
    *out = nullptr;
    xenos_graph_t *gp = nullptr;
    xenos_status_t st = xenos_graph_create(nullptr, &gp);
    if (st != XENOS_OK) return st;
    try {
        Graph &g = gp->g;
        bool compiled = false;
        st = load_graph(g, static_cast<const uint8_t *>(host_buf), bytes, &compiled);
        if (st == XENOS_OK && compiled) {
            size_t wsb = 0;
            st = xenos_graph_compile(gp, g.max_batch, g.precision, &wsb);
            if (st == XENOS_OK && workspace_bytes) *workspace_bytes = wsb;
        } else if (st == XENOS_OK && workspace_bytes) *workspace_bytes = 0;
        if (st != XENOS_OK) {
            g_create_err = std::string("xenos_graph_load: ") + g.err;
            delete gp;
            return st;
        }
    } catch (const std::exception &e) {
        g_create_err = std::string("xenos_graph_load: ") + e.what();
        delete gp;
        return XENOS_E_INVALID;
    }
    *out = gp;
    return XENOS_OK;
}

xenos_status_t xenos_graph_bind(xenos_graph_t *gp, void *workspace_dev, size_t bytes, void *cuda_stream) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state < ST_COMPILED) return fail(g, XENOS_E_STATE, "bind before compile");
    if (!workspace_dev) return fail(g, XENOS_E_WORKSPACE, "bind: workspace is NULL");
    if (bytes < g.workspace_bytes) return fail(g, XENOS_E_WORKSPACE, "bind: workspace too small");
    if (((uintptr_t)workspace_dev & 255u) != 0) return fail(g, XENOS_E_WORKSPACE, "bind: workspace must be 256-byte aligned");
    xenos_status_t st = runtime_bind(g, workspace_dev, bytes, cuda_stream);
    if (st == XENOS_OK) g.state = ST_BOUND;
    return st;
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_run(xenos_graph_t *gp, int32_t batch, const void *const *inputs_dev,
                               void *const *outputs_dev, void *cuda_stream) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state != ST_BOUND) return fail(g, XENOS_E_STATE, "run before bind");
    if (xenos_status_t st = check_run_args(g, "run", batch, inputs_dev, outputs_dev)) return st;
    return runtime_run(g, batch, inputs_dev, outputs_dev, cuda_stream);
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_profile(xenos_graph_t *gp, int32_t batch, const void *const *inputs_dev,
                                   void *const *outputs_dev, void *cuda_stream, float *ms_per_launch,
                                   int32_t n_launches) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state != ST_BOUND) return fail(g, XENOS_E_STATE, "profile before bind");
    if (xenos_status_t st = check_run_args(g, "profile", batch, inputs_dev, outputs_dev)) return st;
    if (!ms_per_launch) return fail(g, XENOS_E_INVALID, "profile: NULL pointer");
    if (n_launches != (int32_t)g.launches.size()) return fail(g, XENOS_E_INVALID, "profile: n_launches must equal xenos_graph_launch_count");
    return runtime_run(g, batch, inputs_dev, outputs_dev, cuda_stream, ms_per_launch);
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_status(xenos_graph_t *gp, void *cuda_stream) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state != ST_BOUND) return fail(g, XENOS_E_STATE, "status before bind");
    return runtime_status(g, cuda_stream);
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_selftest_wait_expiry(xenos_graph_t *gp, void *cuda_stream) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state != ST_BOUND) return fail(g, XENOS_E_STATE, "selftest before bind");
    return runtime_selftest_wait_expiry(g, cuda_stream);
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_get_plan(const xenos_graph_t *gp, char *json, size_t cap, size_t *needed) {
    if (!gp) return XENOS_E_INVALID;
    const Graph &g = gp->g;
    if (g.state < ST_COMPILED) return fail(g, XENOS_E_STATE, "get_plan before compile");
    if (!needed) return fail(g, XENOS_E_INVALID, "get_plan: needed is NULL");
    *needed = g.plan_json.size() + 1;
    if (json && cap > 0) {
        size_t n = g.plan_json.size() < cap - 1 ? g.plan_json.size() : cap - 1;
        std::memcpy(json, g.plan_json.data(), n);
        json[n] = '\0';
    }
    return XENOS_OK;
}

xenos_status_t xenos_graph_launch_count(const xenos_graph_t *gp, int32_t *launches) {
    if (!gp) return XENOS_E_INVALID;
    const Graph &g = gp->g;
    if (g.state < ST_COMPILED) return fail(g, XENOS_E_STATE, "launch_count before compile");
    if (!launches) return fail(g, XENOS_E_INVALID, "launch_count: NULL");
    *launches = (int32_t)g.launches.size();
    return XENOS_OK;
}

xenos_status_t xenos_graph_run_builtin_scratch(xenos_graph_t *gp, int32_t batch, const void *const *inputs_dev,
                                               void *const *outputs_dev, void *cuda_stream) {
    if (!gp) return XENOS_E_INVALID;
    XENOS_GUARD_BEGIN
    Graph &g = gp->g;
    if (g.state < ST_COMPILED) return fail(g, XENOS_E_STATE, "run_builtin_scratch before compile");
    if (xenos_status_t st = check_run_args(g, "run_builtin_scratch", batch, inputs_dev, outputs_dev)) return st;
    if (g.workspace_bytes > runtime_builtin_scratch_bytes())
        return fail(g, XENOS_E_WORKSPACE,
                    "run_builtin_scratch: this graph needs " + std::to_string(g.workspace_bytes) +
                        " workspace bytes but the built-in scratch holds only " +
                        std::to_string(runtime_builtin_scratch_bytes()) + "; use xenos_graph_bind with your own buffer");
    return runtime_run_builtin(g, batch, inputs_dev, outputs_dev, cuda_stream);
    XENOS_GUARD_END(gp)
}

xenos_status_t xenos_graph_destroy(xenos_graph_t *gp) {
    if (!gp) return XENOS_E_INVALID;
    runtime_free_builtin(gp->g);
    runtime_free(gp->g);
    delete gp;
    return XENOS_OK;
}

const char *xenos_last_error(const xenos_graph_t *gp) {
    if (!gp) return g_create_err.c_str();
    return gp->g.err.c_str();
}

}  // extern "C"
