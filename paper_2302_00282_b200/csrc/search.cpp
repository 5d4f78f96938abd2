// Profiling-driven split search: Algorithm 1 of the Xenos paper ("Enumerating Partition Schemes", Section 5)
// restated for one GPU.  The paper enumerates the partition schemes of an operator over the devices, profiles
// each on the hardware and keeps the fastest.  Here the schemes are the split plans of every chain (output-channel
// parts, reduction parts; output-channel / row / column parts for the fp32 CUDA-core chain), the PROFILING step
// is a timed run of a trial plan on the caller's device buffers, and the chains of a graph are searched together:
// a chain's time does not depend on how the other chains are split, so trial t carries candidate t of every chain.
#include <algorithm>
#include <cstdio>
#include <limits>
#include <set>
#include <string>
#include <vector>

#include "graph.hpp"

namespace xenos {

namespace {

struct Cand {
    SplitRequest rq;      // rq.user == false: the planner's own choice (no request)
    std::string label;
};

Graph clone_unbound(const Graph &g) {
    Graph c = g;
    c.ws = nullptr; c.rt = nullptr; c.rt_builtin = nullptr;
    c.err.clear();
    return c;
}

bool compiles_with(const Graph &g, int key, const SplitRequest &rq, int max_batch, int precision) {
    Graph t = clone_unbound(g);
    t.split_requests.push_back({key, rq});
    return compile_graph(t, max_batch, precision) == XENOS_OK;
}

SplitRequest make_rq(int outc, int h, int w, int k) {
    SplitRequest r;
    r.outc = outc; r.h = h; r.w = w; r.k = k; r.user = true;
    return r;
}

}  // namespace

xenos_status_t search_splits(Graph &g, int max_batch, int precision, void *ws, size_t ws_bytes, const void *const *in,
                             void *const *out, void *stream, int max_trials, int repeats, std::string &report) {
    Graph base = clone_unbound(g);
    xenos_status_t st = compile_graph(base, max_batch, precision);
    if (st != XENOS_OK) return fail(g, st, base.err);
    const int nc = (int)base.chains.size();
    std::vector<int> key(nc, -1);
    std::vector<std::vector<Cand>> cands(nc);
    for (int ci = 0; ci < nc; ++ci) {
        const Chain &ch = base.chains[ci];
        key[ci] = base.nodes[ch.nodes.back()].out;
        Cand autoc;
        autoc.label = ch.split.user ? "as requested" : "planner";
        cands[ci].push_back(autoc);
        if (ch.split.user || ch.launches.size() != 1) continue;      // a fixed request is not searched
        const Launch &L = base.launches[ch.launches[0]];
        std::vector<Cand> more;
        auto add = [&](const SplitRequest &rq, const std::string &label) { Cand c; c.rq = rq; c.label = label; more.push_back(c); };
        if (L.kind == LK_GEMM) {
            const bool can_k = ((L.seg[0].mode == AM_GATHER && (L.map_mode == MAP_FLAT || L.a_tma == 2)) || L.seg[0].mode == AM_DW) &&
                               L.seg[1].mode == AM_NONE && L.epi == EPI_STORE;
            add(make_rq(L.n_tiles * 2, 0, 0, 1), "outc x2");
            if (L.n_tiles > 1) add(make_rq((L.n_tiles + 1) / 2, 0, 0, 1), "outc /2");
            if (can_k) {
                for (int k : {2, 4, 8})
                    if (k != L.ksplit && 2 * k <= L.kblocks) add(make_rq(L.n_tiles, 0, 0, k), "k " + std::to_string(k));
                if (L.ksplit > 1) add(make_rq(L.n_tiles, 0, 0, 1), "k 1");
            }
        } else if (L.kind == LK_F32_CONV_CONV_POOL) {
            // the two orders of Section 4.2.1 and mixtures: output channels first, rows / columns first
            for (int oc : {1, 2, 4, 8})
                for (int hw : {1, 2, 4, 8, 16})
                    if (!(oc == L.parts_outc && hw == L.tiles_h && hw == L.tiles_w))
                        add(make_rq(oc, hw, hw, 1), "outc " + std::to_string(oc) + " rows " + std::to_string(hw) + " cols " + std::to_string(hw));
        }
        for (const Cand &c : more)
            if ((int)cands[ci].size() < max_trials && compiles_with(g, key[ci], c.rq, max_batch, precision)) cands[ci].push_back(c);
    }
    size_t trials = 1;
    for (int ci = 0; ci < nc; ++ci) trials = std::max(trials, cands[ci].size());
    const double inf = std::numeric_limits<double>::infinity();
    std::vector<std::vector<double>> ms(nc);
    for (int ci = 0; ci < nc; ++ci) ms[ci].assign(cands[ci].size(), inf);
    for (size_t t = 0; t < trials; ++t) {
        Graph trial = clone_unbound(g);
        for (int ci = 0; ci < nc; ++ci)
            if (t > 0 && t < cands[ci].size()) trial.split_requests.push_back({key[ci], cands[ci][t].rq});
        st = compile_graph(trial, max_batch, precision);
        if (st != XENOS_OK) return fail(g, st, "search: trial plan does not compile: " + trial.err);
        if (trial.workspace_bytes > ws_bytes)
            return fail(g, XENOS_E_WORKSPACE, "search: a trial plan needs " + std::to_string(trial.workspace_bytes) + " workspace bytes");
        if ((int)trial.chains.size() != nc) return fail(g, XENOS_E_INVALID, "internal: chains changed between trials");
        st = runtime_bind(trial, ws, ws_bytes, stream);
        std::vector<float> per(trial.launches.size()), acc(trial.launches.size(), 0.0f);
        for (int r = 0; r <= repeats && st == XENOS_OK; ++r) {      // the first run warms up
            st = runtime_run(trial, max_batch, in, out, stream, per.data());
            if (r > 0) for (size_t i = 0; i < per.size(); ++i) acc[i] += per[i];
        }
        if (st == XENOS_OK) st = runtime_status(trial, stream);
        std::string err = trial.err;
        runtime_free(trial);
        if (st != XENOS_OK) return fail(g, st, "search: " + err);
        for (int ci = 0; ci < nc; ++ci) {
            double sum = 0;
            for (int li : trial.chains[ci].launches) sum += acc[li] / repeats;
            const size_t idx = t < cands[ci].size() ? t : 0;
            ms[ci][idx] = std::min(ms[ci][idx], sum);
        }
    }
    // keep the fastest scheme of every chain; it becomes a split request of the graph
    report = "{\"trials\":" + std::to_string(trials) + ",\"chains\":[";
    for (int ci = 0; ci < nc; ++ci) {
        size_t best = 0;
        for (size_t i = 1; i < cands[ci].size(); ++i)
            if (ms[ci][i] < ms[ci][best]) best = i;
        if (best > 0) g.split_requests.push_back({key[ci], cands[ci][best].rq});
        if (ci) report += ",";
        report += "{\"id\":" + std::to_string(ci) + ",\"tensor\":" + std::to_string(key[ci]) + ",\"chosen\":" + std::to_string(best) + ",\"candidates\":[";
        for (size_t i = 0; i < cands[ci].size(); ++i) {
            char buf[64];
            snprintf(buf, sizeof buf, "%.3f", ms[ci][i] * 1e3);
            const SplitRequest &r = cands[ci][i].rq;
            if (i) report += ",";
            report += "{\"label\":\"" + cands[ci][i].label + "\",\"parts_outc\":" + std::to_string(r.user ? r.outc : 0) +
                      ",\"parts_h\":" + std::to_string(r.user ? r.h : 0) + ",\"parts_w\":" + std::to_string(r.user ? r.w : 0) +
                      ",\"parts_k\":" + std::to_string(r.user ? r.k : 0) + ",\"us\":" + buf + "}";
        }
        report += "]}";
    }
    report += "]}";
    return XENOS_OK;
}

}  // namespace xenos
