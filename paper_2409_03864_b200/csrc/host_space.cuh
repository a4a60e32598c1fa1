// A search space stated by the caller, in the form of the tuning-parameter listing of the paper's Case Study 5:
// every parameter of the tile configuration gets a range, and constraints relate the parameters to each other and
// to the problem -- "the tile size divides its dimension", "vectorise only if the inner trip count divides".
//
//   space      := statement (';' statement)*
//   statement  := param 'in' '{' int (',' int)* '}'            a list of values
//              |  param 'in' int '..' int ['step' int]         an inclusive range
//              |  'require' expr                               keep a candidate only if expr holds
//              |  param '==' int 'only' 'if' expr              candidates with that value must satisfy expr
//   expr       := C-like integer expression over the parameters (tile_m tile_n tile_k stages cta_pair split_k store_mode
//                 raster k_stagger fit), the problem (M N K transA transB num_kb) and integers, with
//                 + - * / % == != < <= > >= && || ! and parentheses
//
// Parameters the text does not mention stay 0 ("choose for me") and are filled in by the library's rules; the
// hardware's own constraints (shared memory, tensor memory, layout divisibility) are applied afterwards.
#pragma once
#include "host_plan.cuh"

namespace {

struct SpaceParam { std::string name; std::vector<long long> values; };
struct SpaceRule { bool conditional = false; std::string param; long long value = 0; std::string expr; };
struct SearchSpace {
    std::vector<SpaceParam> params;
    std::vector<SpaceRule> rules;
};

const char* const kSpaceParamNames[] = {"tile_m", "tile_n", "tile_k", "stages", "cta_pair", "split_k", "store_mode", "raster",
                                        "k_stagger", "fit"};

int* space_field(tdx_config* c, const std::string& n) {
    if (n == "tile_m") return &c->tile_m;
    if (n == "tile_n") return &c->tile_n;
    if (n == "tile_k") return &c->tile_k;
    if (n == "stages") return &c->stages;
    if (n == "cta_pair") return &c->cta_pair;
    if (n == "split_k") return &c->split_k;
    if (n == "store_mode") return &c->store_mode;
    if (n == "raster") return &c->raster;
    if (n == "k_stagger") return &c->k_stagger;
    if (n == "fit") return &c->fit;
    return nullptr;
}

// ---- a small recursive-descent evaluator of integer expressions
struct ExprEval {
    const char* s;
    const std::map<std::string, long long>* vars;
    std::string err;

    void skip() { while (*s == ' ' || *s == '\t' || *s == '\n') ++s; }
    bool eat(const char* tok) {
        skip();
        const size_t n = std::strlen(tok);
        if (std::strncmp(s, tok, n) != 0) return false;
        s += n;
        return true;
    }
    long long primary() {
        skip();
        if (*s == '(') {
            ++s;
            const long long v = lor();
            if (!eat(")")) err = "missing ')'";
            return v;
        }
        if (*s == '!' && s[1] != '=') { ++s; return !primary(); }
        if (*s == '-') { ++s; return -primary(); }
        if (*s >= '0' && *s <= '9') {
            char* end;
            const long long v = std::strtoll(s, &end, 10);
            s = end;
            return v;
        }
        if ((*s >= 'a' && *s <= 'z') || (*s >= 'A' && *s <= 'Z') || *s == '_') {
            std::string id;
            while ((*s >= 'a' && *s <= 'z') || (*s >= 'A' && *s <= 'Z') || (*s >= '0' && *s <= '9') || *s == '_') id += *s++;
            auto it = vars->find(id);
            if (it == vars->end()) { err = "unknown name '" + id + "'"; return 0; }
            return it->second;
        }
        err = std::string("unexpected '") + (*s ? std::string(1, *s) : std::string("end of text")) + "'";
        return 0;
    }
    long long mul() {
        long long v = primary();
        for (;;) {
            skip();
            if (*s == '*') { ++s; v *= primary(); }
            else if (*s == '/') { ++s; const long long d = primary(); if (!err.empty()) return 0; if (d == 0) { err = "division by zero"; return 0; } v /= d; }
            else if (*s == '%') { ++s; const long long d = primary(); if (!err.empty()) return 0; if (d == 0) { err = "division by zero"; return 0; } v %= d; }
            else return v;
            if (!err.empty()) return 0;
        }
    }
    long long add() {
        long long v = mul();
        for (;;) {
            skip();
            if (*s == '+') { ++s; v += mul(); }
            else if (*s == '-') { ++s; v -= mul(); }
            else return v;
            if (!err.empty()) return 0;
        }
    }
    long long cmp() {
        long long v = add();
        for (;;) {
            if (eat("==")) v = (v == add());
            else if (eat("!=")) v = (v != add());
            else if (eat("<=")) v = (v <= add());
            else if (eat(">=")) v = (v >= add());
            else if (eat("<")) v = (v < add());
            else if (eat(">")) v = (v > add());
            else return v;
            if (!err.empty()) return 0;
        }
    }
    long long land() {
        long long v = cmp();
        while (err.empty() && eat("&&")) { const long long r = cmp(); v = (v && r); }
        return v;
    }
    long long lor() {
        long long v = land();
        while (err.empty() && eat("||")) { const long long r = land(); v = (v || r); }
        return v;
    }
};

// value of `expr` under `vars`; false + message on a syntax error or an unknown name
bool eval_space_expr(const std::string& expr, const std::map<std::string, long long>& vars, long long* out, std::string* err) {
    ExprEval e{expr.c_str(), &vars, ""};
    const long long v = e.lor();
    e.skip();
    if (e.err.empty() && *e.s != '\0') e.err = std::string("unexpected '") + *e.s + "'";
    if (!e.err.empty()) { *err = e.err + " in \"" + expr + "\""; return false; }
    *out = v;
    return true;
}

std::string space_trim(const std::string& t) {
    size_t a = 0, b = t.size();
    while (a < b && (t[a] == ' ' || t[a] == '\t' || t[a] == '\n')) ++a;
    while (b > a && (t[b - 1] == ' ' || t[b - 1] == '\t' || t[b - 1] == '\n')) --b;
    return t.substr(a, b - a);
}

bool parse_search_space(const char* text, SearchSpace* out, std::string* err) {
    std::string all(text ? text : "");
    size_t pos = 0;
    while (pos <= all.size()) {
        const size_t semi = all.find(';', pos);
        const std::string st = space_trim(all.substr(pos, semi == std::string::npos ? std::string::npos : semi - pos));
        pos = semi == std::string::npos ? all.size() + 1 : semi + 1;
        if (st.empty()) continue;
        if (st.compare(0, 8, "require ") == 0) {
            SpaceRule r;
            r.expr = space_trim(st.substr(8));
            out->rules.push_back(r);
            continue;
        }
        const size_t only = st.find(" only if ");
        if (only != std::string::npos) {
            const size_t eq = st.find("==");
            if (eq == std::string::npos || eq > only) { *err = "expected '<param> == <value> only if <expr>' in \"" + st + "\""; return false; }
            SpaceRule r;
            r.conditional = true;
            r.param = space_trim(st.substr(0, eq));
            tdx_config probe;
            if (space_field(&probe, r.param) == nullptr) { *err = "unknown parameter '" + r.param + "'"; return false; }
            r.value = std::strtoll(st.c_str() + eq + 2, nullptr, 10);
            r.expr = space_trim(st.substr(only + 9));
            out->rules.push_back(r);
            continue;
        }
        const size_t in = st.find(" in ");
        if (in == std::string::npos) { *err = "cannot read statement \"" + st + "\""; return false; }
        SpaceParam p;
        p.name = space_trim(st.substr(0, in));
        tdx_config probe;
        if (space_field(&probe, p.name) == nullptr) { *err = "unknown parameter '" + p.name + "'"; return false; }
        for (const auto& q : out->params)
            if (q.name == p.name) { *err = "parameter '" + p.name + "' is given twice"; return false; }
        const std::string rhs = space_trim(st.substr(in + 4));
        if (!rhs.empty() && rhs[0] == '{') {
            const size_t close = rhs.find('}');
            if (close == std::string::npos) { *err = "missing '}' in \"" + st + "\""; return false; }
            const char* s = rhs.c_str() + 1;
            const char* end = rhs.c_str() + close;
            while (s < end) {
                char* next;
                const long long v = std::strtoll(s, &next, 10);
                if (next == s) { *err = "expected an integer in \"" + st + "\""; return false; }
                p.values.push_back(v);
                s = next;
                while (s < end && (*s == ',' || *s == ' ')) ++s;
            }
        } else {
            const size_t dots = rhs.find("..");
            if (dots == std::string::npos) { *err = "expected '{...}' or 'lo..hi' in \"" + st + "\""; return false; }
            const long long lo = std::strtoll(rhs.c_str(), nullptr, 10);
            const long long hi = std::strtoll(rhs.c_str() + dots + 2, nullptr, 10);
            long long step = 1;
            const size_t sp = rhs.find("step");
            if (sp != std::string::npos) step = std::strtoll(rhs.c_str() + sp + 4, nullptr, 10);
            if (step < 1 || hi < lo || (hi - lo) / step > 4096) { *err = "bad range in \"" + st + "\""; return false; }
            for (long long v = lo; v <= hi; v += step) p.values.push_back(v);
        }
        if (p.values.empty()) { *err = "empty range for '" + p.name + "'"; return false; }
        out->params.push_back(p);
    }
    return true;
}

// The candidates of `space` for one GEMM: the cross product of the ranges (`n_product`), minus what the stated rules
// exclude (`n_after_rules`), each then completed by resolve() and kept if statically feasible; duplicates dropped.
template <typename Resolve>
bool enumerate_search_space(const SearchSpace& space, const GemmProblem& g, Resolve&& resolve, std::vector<tdx_config>* out,
                            long long* n_product, long long* n_after_rules, std::string* err) {
    long long total = 1;
    for (const auto& p : space.params) {
        total *= static_cast<long long>(p.values.size());
        if (total > (1LL << 20)) { *err = "search space larger than 2^20 candidates"; return false; }
    }
    *n_product = total;
    *n_after_rules = 0;
    std::map<std::string, long long> vars;
    vars["M"] = g.M; vars["N"] = g.N; vars["K"] = g.K; vars["transA"] = g.transA; vars["transB"] = g.transB;
    vars["num_kb"] = ceil_div(g.K, 64);
    std::vector<size_t> idx(space.params.size(), 0);
    for (long long n = 0; n < total; ++n) {
        tdx_config c;
        std::memset(&c, 0, sizeof c);
        c.kernel = TDX_KERNEL_UMMA;
        for (const char* name : kSpaceParamNames) vars[name] = 0;
        for (size_t i = 0; i < space.params.size(); ++i) {
            const long long v = space.params[i].values[idx[i]];
            *space_field(&c, space.params[i].name) = static_cast<int>(v);
            vars[space.params[i].name] = v;
        }
        bool keep = true;
        for (const auto& r : space.rules) {
            if (r.conditional && vars[r.param] != r.value) continue;
            long long v = 0;
            if (!eval_space_expr(r.expr, vars, &v, err)) return false;
            if (!v) { keep = false; break; }
        }
        if (keep) {
            ++*n_after_rules;
            tdx_config full;
            if (resolve(c, &full)) {
                bool dup = false;
                for (const auto& o : *out)
                    if (std::memcmp(&o, &full, sizeof full) == 0) { dup = true; break; }
                if (!dup) out->push_back(full);
            }
        }
        for (size_t i = 0; i < idx.size(); ++i) {            // next point of the cross product
            if (++idx[i] < space.params[i].values.size()) break;
            idx[i] = 0;
        }
    }
    return true;
}

}  // namespace
