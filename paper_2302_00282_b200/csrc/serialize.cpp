// Graph image: the optimised model as one host byte string that can be stored and loaded again (Section 6 of the
// Xenos paper: the optimiser hands the runtime an executable of the optimised model; Section 3: it replaces the
// original model file).  The image holds what the plan is a function of: the hardware description, the tensors and
// operators with their parameters, the link and split requests, and the compile options.  Loading it rebuilds the
// graph and, if the saved graph was compiled, compiles it again: planning is deterministic, so the loaded graph's
// plan is byte-identical to the saved one's, and no device address or pointer ever enters the image.
//
// Layout (little-endian): "XENOSIMG" | u32 version | body | u64 FNV-1a of everything before it.
// The body is a sequence of i32 / u64 / f32-array fields in the order written below; every count and index is
// range-checked on load.
#include <cstring>
#include <string>
#include <vector>

#include "graph.hpp"

namespace xenos {

namespace {

constexpr char kMagic[8] = {'X', 'E', 'N', 'O', 'S', 'I', 'M', 'G'};
constexpr uint32_t kVersion = 1;

uint64_t fnv1a(const uint8_t *p, size_t n) {
    uint64_t h = 1469598103934665603ull;
    for (size_t i = 0; i < n; ++i) { h ^= p[i]; h *= 1099511628211ull; }
    return h;
}

struct Writer {
    std::vector<uint8_t> b;
    void raw(const void *p, size_t n) { const uint8_t *q = static_cast<const uint8_t *>(p); b.insert(b.end(), q, q + n); }
    void i32(int32_t v) { raw(&v, 4); }
    void u64(uint64_t v) { raw(&v, 8); }
    void f32(float v) { raw(&v, 4); }
    void ints(const std::vector<int> &v) { u64(v.size()); for (int x : v) i32(x); }
    void floats(const std::vector<float> &v) { u64(v.size()); if (!v.empty()) raw(v.data(), v.size() * 4); }
};

struct Reader {
    const uint8_t *p;
    size_t n, at = 0;
    bool bad = false;
    bool take(void *dst, size_t k) {
        if (bad || k > n - at) { bad = true; return false; }
        std::memcpy(dst, p + at, k);
        at += k;
        return true;
    }
    int32_t i32() { int32_t v = 0; take(&v, 4); return v; }
    uint64_t u64() { uint64_t v = 0; take(&v, 8); return v; }
    float f32() { float v = 0; take(&v, 4); return v; }
    // a count of elements of `elem` bytes that the rest of the image can hold
    size_t count(size_t elem) {
        uint64_t c = u64();
        if (bad || c > (n - at) / (elem ? elem : 1)) { bad = true; return 0; }
        return (size_t)c;
    }
    std::vector<int> ints() { size_t c = count(4); std::vector<int> v(c); for (size_t i = 0; i < c && !bad; ++i) v[i] = i32(); return v; }
    std::vector<float> floats() { size_t c = count(4); std::vector<float> v(c); if (c) take(v.data(), c * 4); return v; }
};

}  // namespace

void save_graph(const Graph &g, std::vector<uint8_t> &out) {
    Writer w;
    w.raw(kMagic, 8);
    w.raw(&kVersion, 4);
    w.i32(g.hw.sm_count); w.i32(g.hw.smem_bytes_per_cta); w.i32(g.hw.tmem_columns); w.u64((uint64_t)g.hw.l2_bytes);
    w.u64(g.tensors.size());
    for (const Tensor &t : g.tensors) {
        w.i32(t.c); w.i32(t.h); w.i32(t.w); w.i32(t.is_vec); w.i32(t.producer); w.ints(t.consumers);
        w.i32(t.input_slot); w.i32(t.output_slot); w.i32(t.io_dtype); w.i32(t.io_layout);
    }
    w.u64(g.ops.size());
    for (const Op &o : g.ops) {
        w.i32(o.kind); w.i32(o.cout); w.i32(o.k); w.i32(o.stride); w.i32(o.pad); w.i32(o.groups); w.i32(o.act);
        w.ints(o.in); w.i32(o.out);
        w.floats(o.w); w.floats(o.bias); w.floats(o.gamma); w.floats(o.beta); w.floats(o.mean); w.floats(o.var);
        w.f32(o.eps); w.i32(o.has_bias); w.i32(o.has_bn);
    }
    w.ints(g.inputs); w.ints(g.outputs);
    w.i32(g.link_auto);
    w.u64(g.link_requests.size());
    for (const LinkRequest &r : g.link_requests) w.ints(r.ops);
    w.u64(g.split_requests.size());
    for (const auto &r : g.split_requests) {
        w.i32(r.first); w.i32(r.second.outc); w.i32(r.second.h); w.i32(r.second.w); w.i32(r.second.k); w.i32(r.second.user);
    }
    w.i32(g.state >= ST_COMPILED ? 1 : 0); w.i32(g.precision); w.i32(g.max_batch);
    w.u64(fnv1a(w.b.data(), w.b.size()));
    out.swap(w.b);
}

// Fills `g` (a fresh graph) from an image.  Returns XENOS_E_INVALID for anything that is not an intact image of this
// version; on success *compiled tells whether the saved graph was compiled (g.precision / g.max_batch then hold the
// options to compile with).
xenos_status_t load_graph(Graph &g, const uint8_t *buf, size_t bytes, bool *compiled) {
    if (!buf || bytes < 8 + 4 + 8) return fail(g, XENOS_E_INVALID, "load: the buffer is too short for a graph image");
    if (std::memcmp(buf, kMagic, 8) != 0) return fail(g, XENOS_E_INVALID, "load: not a graph image");
    uint64_t sum = 0;
    std::memcpy(&sum, buf + bytes - 8, 8);
    if (sum != fnv1a(buf, bytes - 8)) return fail(g, XENOS_E_INVALID, "load: checksum mismatch (truncated or altered image)");
    Reader r{buf, bytes - 8};
    r.at = 8;
    uint32_t ver = 0;
    r.take(&ver, 4);
    if (ver != kVersion) return fail(g, XENOS_E_INVALID, "load: image version " + std::to_string(ver) + " is not supported");
    g.hw.sm_count = r.i32(); g.hw.smem_bytes_per_cta = r.i32(); g.hw.tmem_columns = r.i32(); g.hw.l2_bytes = (int64_t)r.u64();
    if (g.hw.sm_count < 1 || g.hw.smem_bytes_per_cta < 48 * 1024 || g.hw.tmem_columns < 32 || g.hw.tmem_columns > 512 || g.hw.l2_bytes < 0)
        return fail(g, XENOS_E_INVALID, "load: hardware info out of range");
    const size_t nt = r.count(40);
    g.tensors.assign(nt, Tensor());
    for (Tensor &t : g.tensors) {
        t.c = r.i32(); t.h = r.i32(); t.w = r.i32(); t.is_vec = r.i32() != 0; t.producer = r.i32(); t.consumers = r.ints();
        t.input_slot = r.i32(); t.output_slot = r.i32(); t.io_dtype = r.i32(); t.io_layout = r.i32();
    }
    const size_t no = r.count(40);
    g.ops.assign(no, Op());
    for (Op &o : g.ops) {
        o.kind = r.i32(); o.cout = r.i32(); o.k = r.i32(); o.stride = r.i32(); o.pad = r.i32(); o.groups = r.i32(); o.act = r.i32();
        o.in = r.ints(); o.out = r.i32();
        o.w = r.floats(); o.bias = r.floats(); o.gamma = r.floats(); o.beta = r.floats(); o.mean = r.floats(); o.var = r.floats();
        o.eps = r.f32(); o.has_bias = r.i32() != 0; o.has_bn = r.i32() != 0;
    }
    g.inputs = r.ints(); g.outputs = r.ints();
    g.link_auto = r.i32() != 0;
    const size_t nl = r.count(8);
    g.link_requests.assign(nl, LinkRequest());
    for (LinkRequest &q : g.link_requests) q.ops = r.ints();
    const size_t ns = r.count(24);
    g.split_requests.clear();
    for (size_t i = 0; i < ns && !r.bad; ++i) {
        SplitRequest q;
        const int key = r.i32();
        q.outc = r.i32(); q.h = r.i32(); q.w = r.i32(); q.k = r.i32(); q.user = r.i32() != 0;
        g.split_requests.push_back({key, q});
    }
    const bool was_compiled = r.i32() != 0;
    g.precision = r.i32(); g.max_batch = r.i32();
    if (r.bad || r.at != r.n) return fail(g, XENOS_E_INVALID, "load: the image's fields do not fill it exactly");
    // every index names something that exists (the passes index without checking)
    const int T = (int)g.tensors.size(), O = (int)g.ops.size();
    auto tid = [&](int x) { return x >= 0 && x < T; };
    for (const Tensor &t : g.tensors) {
        if (t.producer < -1 || t.producer >= O) return fail(g, XENOS_E_INVALID, "load: tensor producer out of range");
        for (int c : t.consumers) if (c < 0 || c >= O) return fail(g, XENOS_E_INVALID, "load: tensor consumer out of range");
        if (t.c < 1 || t.h < 0 || t.w < 0) return fail(g, XENOS_E_INVALID, "load: tensor extent out of range");
    }
    for (const Op &o : g.ops) {
        if (!tid(o.out)) return fail(g, XENOS_E_INVALID, "load: operator output out of range");
        for (int x : o.in) if (!tid(x)) return fail(g, XENOS_E_INVALID, "load: operator input out of range");
    }
    for (int x : g.inputs) if (!tid(x)) return fail(g, XENOS_E_INVALID, "load: graph input out of range");
    for (int x : g.outputs) if (!tid(x)) return fail(g, XENOS_E_INVALID, "load: graph output out of range");
    for (const LinkRequest &q : g.link_requests) for (int x : q.ops) if (!tid(x)) return fail(g, XENOS_E_INVALID, "load: link request out of range");
    for (const auto &q : g.split_requests) if (!tid(q.first)) return fail(g, XENOS_E_INVALID, "load: split request out of range");
    g.state = ST_BUILD;
    *compiled = was_compiled;
    return XENOS_OK;
}

}  // namespace xenos
