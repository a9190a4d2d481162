// The steps of Algorithm 3 around the search, for one expression: sketches from a (source,
// erroneous) pair of expressions, the per-index constraints, the batched search and the
// stitching of the solution back into the expression.  Host code only; it uses the library
// through its own C ABI (include/xp.h) and nothing else.
#include <chrono>
#include <new>
#include <string>
#include <vector>

#include "xp.h"

namespace xp { xp_status set_error(xp_status st, const char* msg); }      // records the calling thread's error message

namespace {

const char* const kOpText[] = {"+", "-", "*", "/", "%", "<", "<=", "==", "!=", "min", "max", "&&", "||", "<<", ">>"};

// first[i]: index of the first instruction of the subtree whose root is instruction i.
bool subtree_starts(const xp_instr* code, int n, std::vector<int>* first) {
    std::vector<int> st;
    first->assign(n, 0);
    for (int i = 0; i < n; ++i) {
        if (code[i].kind == XP_I_OP) {
            if (st.size() < 2) return false;
            st.pop_back();
            (*first)[i] = st.back();
            st.back() = (*first)[i];
        } else {
            (*first)[i] = i;
            st.push_back(i);
        }
    }
    return st.size() == 1;
}

std::string text_of(const xp_instr* code, int n, const std::vector<std::string>& names) {
    std::vector<std::string> st;
    for (int i = 0; i < n; ++i) {
        const xp_instr& c = code[i];
        if (c.kind == XP_I_VAR) st.push_back(c.arg >= 0 && c.arg < (int)names.size() ? names[c.arg] : "v" + std::to_string(c.arg));
        else if (c.kind == XP_I_CONST) st.push_back(std::to_string((long long)c.value));
        else if (c.kind == XP_I_HOLE) st.push_back("HOLE");
        else {
            const std::string r = st.back(); st.pop_back();
            const std::string l = st.back(); st.pop_back();
            const bool call = c.arg == XP_OP_MIN || c.arg == XP_OP_MAX;
            st.push_back(call ? std::string(kOpText[c.arg]) + "(" + l + "," + r + ")" : "(" + l + kOpText[c.arg] + r + ")");
        }
    }
    return st.empty() ? std::string() : st.back();
}

}  // namespace

struct xp_pair_result {
    xp_pair_view v;
    std::string hole_text, sketch_text, stitched_text;
    std::vector<xp_instr> stitched;
};

extern "C" xp_status xp_pair_result_get(const xp_pair_result* r, xp_pair_view* out) {
    if (!r || !out) return XP_ERR_INVALID_ARG;
    *out = r->v;
    out->hole_text = r->hole_text.c_str();
    out->sketch_text = r->sketch_text.c_str();
    out->stitched_text = r->stitched_text.c_str();
    out->stitched_code = r->stitched.data();
    out->stitched_len = (int32_t)r->stitched.size();
    return XP_OK;
}

extern "C" void xp_pair_result_free(xp_pair_result* r) { delete r; }

extern "C" xp_status xp_repair_pair(const xp_grammar* g, const xp_pair_desc* d, xp_pair_result** out) {
    if (!g || !d || !out || !d->source || !d->erroneous || d->source_len < 1 || d->erroneous_len < 1)
        return xp::set_error(XP_ERR_INVALID_ARG, "xp_repair_pair: null or empty argument");
    *out = nullptr;
    const int ne = d->erroneous_len;
    std::vector<int> first;
    if (ne > XP_MAX_CODE || !subtree_starts(d->erroneous, ne, &first)) return xp::set_error(XP_ERR_SKETCH, "xp_repair_pair: malformed erroneous expression");
    for (int i = 0; i < ne; ++i) if (d->erroneous[i].kind == XP_I_HOLE) return xp::set_error(XP_ERR_SKETCH, "xp_repair_pair: the erroneous expression contains a hole");
    // CreateSMTQuery: S_s over the transformed program's variables
    std::vector<xp_instr> spec;
    for (int i = 0; i < d->source_len; ++i) {
        const xp_instr& c = d->source[i];
        if (c.kind == XP_I_HOLE) return xp::set_error(XP_ERR_SKETCH, "xp_repair_pair: the source expression contains a hole");
        if (c.kind == XP_I_VAR && d->var_map) {
            if (c.arg < 0 || c.arg >= d->n_source_vars || !d->var_map[c.arg] || !d->var_map_len || d->var_map_len[c.arg] < 1)
                return xp::set_error(XP_ERR_SKETCH, "xp_repair_pair: a source variable has no expression in var_map");
            spec.insert(spec.end(), d->var_map[c.arg], d->var_map[c.arg] + d->var_map_len[c.arg]);
        } else spec.push_back(c);
    }
    if (spec.size() > (size_t)XP_MAX_CODE) return xp::set_error(XP_ERR_SKETCH, "xp_repair_pair: the source expression over the target variables is longer than XP_MAX_CODE");
    // GenerateCodeSketch: one sketch per node of S_e
    std::vector<std::vector<xp_instr>> ctx(ne);
    std::vector<xp_hole_desc> holes(ne);
    std::vector<xp_sketch_desc> descs(ne);
    std::vector<const xp_grammar*> grammars(ne, g);
    for (int i = 0; i < ne; ++i) {
        for (int k = 0; k < first[i]; ++k) ctx[i].push_back(d->erroneous[k]);
        xp_instr h;
        h.kind = XP_I_HOLE; h.arg = 0; h.value = 0;
        ctx[i].push_back(h);
        for (int k = i + 1; k < ne; ++k) ctx[i].push_back(d->erroneous[k]);
        xp_hole_desc& hd = holes[i];
        hd = xp_hole_desc();
        hd.start_nt = d->start_nt; hd.max_size = d->max_size;
        hd.ctx_len = ctx[i].size() == 1 ? 0 : (int32_t)ctx[i].size();       // the whole expression taken out: identity context
        hd.ctx = ctx[i].data();
        hd.spec_kind = XP_SPEC_EXPR; hd.spec_len = (int32_t)spec.size(); hd.spec_expr = spec.data();
        xp_sketch_desc& sd = descs[i];
        sd = xp_sketch_desc();
        sd.domain_kind = XP_DOMAIN_BOX; sd.n_holes = 1; sd.holes = &hd;
    }
    // SynthesisCode: the whole ladder of sketches in one batch
    const auto t0 = std::chrono::steady_clock::now();
    std::vector<xp_sketch*> loaded(ne, nullptr);
    xp_status st = xp_sketch_load_batch(grammars.data(), descs.data(), (size_t)ne, loaded.data());
    if (st != XP_OK) return st;
    const auto t1 = std::chrono::steady_clock::now();
    std::vector<xp_result*> results(ne, nullptr);
    st = xp_repair_batch(loaded.data(), (size_t)ne, nullptr, results.data());
    const auto t2 = std::chrono::steady_clock::now();
    xp_pair_result* r = st == XP_OK ? new (std::nothrow) xp_pair_result : nullptr;
    if (st == XP_OK && !r) st = XP_ERR_NOMEM;
    if (st == XP_OK) {
        r->v = xp_pair_view();
        r->v.n_sketches = ne;
        r->v.node_first = r->v.node_last = -1;
        r->v.load_ms = std::chrono::duration<double, std::milli>(t1 - t0).count();
        r->v.search_ms = std::chrono::duration<double, std::milli>(t2 - t1).count();
        int best = -1;
        xp_result_view bv = xp_result_view();
        for (int i = 0; i < ne; ++i) {
            xp_result_view v;
            if (xp_result_get(results[i], 0, &v) != XP_OK) continue;
            for (int k = 1; k <= v.max_size; ++k) r->v.candidates += v.cand_count[k];
            r->v.evals_executed += v.evals_executed;
            if (!v.solved) continue;
            const int len = i - first[i] + 1, best_len = best >= 0 ? best - first[best] + 1 : 0;
            const bool better = best < 0 || v.least_size < bv.least_size ||
                                (v.least_size == bv.least_size && (len < best_len || (len == best_len && first[i] < first[best])));
            if (better) { best = i; bv = v; }
        }
        // StitchBack
        std::vector<std::string> names;
        {   // variable names as the grammar prints them: unrank every leaf once
            char buf[256];
            xp_instr one;
            for (uint64_t k = 0;; ++k) {
                if (xp_grammar_unrank(g, d->start_nt, 1, k, &one, 1, buf, sizeof(buf)) != XP_OK) break;
                if (one.kind == XP_I_VAR) { if ((int)names.size() <= one.arg) names.resize(one.arg + 1); names[one.arg] = buf; }
            }
        }
        if (best >= 0) {
            r->v.solved = 1;
            r->v.node_first = first[best]; r->v.node_last = best;
            r->v.least_size = bv.least_size; r->v.least_rank = bv.least_rank;
            r->hole_text = bv.least_text;
            r->sketch_text = text_of(ctx[best].data(), (int)ctx[best].size(), names);
            for (int k = 0; k < first[best]; ++k) r->stitched.push_back(d->erroneous[k]);
            r->stitched.insert(r->stitched.end(), bv.least_code, bv.least_code + bv.least_len);
            for (int k = best + 1; k < ne; ++k) r->stitched.push_back(d->erroneous[k]);
            r->stitched_text = text_of(r->stitched.data(), (int)r->stitched.size(), names);
        }
        *out = r;
    }
    for (int i = 0; i < ne; ++i) { if (results[i]) xp_result_free(results[i]); if (loaded[i]) xp_sketch_destroy(loaded[i]); }
    return st;
}
