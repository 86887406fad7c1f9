// Schedule descriptor: parser, legality checker and kernel-family matcher (host only).
//
// The checker restates the constraint system of Sec. 3.2 as predicates over a *given* solution:
// instead of asking a solver for ap / dp / lp values it verifies the ones it is handed.
#include "plan.h"

#include <algorithm>
#include <cctype>
#include <set>

namespace cb {
namespace {

bool parse_ref(const std::string &text, TensorRef &ref) {
    size_t p = 0, n = text.size();
    auto skip = [&] { while (p < n && std::isspace((unsigned char)text[p])) ++p; };
    skip();
    size_t s = p;
    while (p < n && (std::isalnum((unsigned char)text[p]) || text[p] == '_')) ++p;
    if (p == s || std::isdigit((unsigned char)text[s])) return false;
    ref.name = text.substr(s, p - s);
    ref.idx.clear();
    skip();
    if (p >= n || text[p] != '[') return false;
    ++p;
    bool want_index = true;
    for (;;) {
        skip();
        if (p >= n) return false;
        if (text[p] == ']') { ++p; break; }
        if (want_index) {
            if (!std::isalpha((unsigned char)text[p])) return false;
            ref.idx.push_back(text[p++]);
            want_index = false;
        } else {
            if (text[p] != ',') return false;
            ++p;
            want_index = true;
        }
    }
    if (want_index && !ref.idx.empty()) return false;      // trailing comma
    skip();
    if (p != n) return false;
    std::set<char> uniq(ref.idx.begin(), ref.idx.end());   // indices of a reference are distinct (Sec. 2.1)
    return uniq.size() == ref.idx.size() && !ref.idx.empty();
}

bool parse_assignment(const std::string &text, TensorRef &lhs, std::vector<TensorRef> &rhs) {
    size_t eq = text.find('=');
    if (eq == std::string::npos || text.find('=', eq + 1) != std::string::npos) return false;
    if (!parse_ref(text.substr(0, eq), lhs)) return false;
    rhs.clear();
    std::string rest = text.substr(eq + 1);
    size_t start = 0;
    for (;;) {
        size_t star = rest.find('*', start);
        TensorRef r;
        if (!parse_ref(rest.substr(start, star == std::string::npos ? std::string::npos : star - start), r))
            return false;
        rhs.push_back(r);
        if (star == std::string::npos) break;
        start = star + 1;
    }
    return true;
}

bool is_permutation(const std::vector<int> &v) {
    std::vector<int> s(v);
    std::sort(s.begin(), s.end());
    for (size_t i = 0; i < s.size(); ++i) if (s[i] != (int)i) return false;
    return true;
}

std::string index_union(const Contraction &c) {
    std::string u;
    for (const TensorRef *r : {&c.lhs, &c.rhs, &c.out})
        for (char x : r->idx) if (u.find(x) == std::string::npos) u.push_back(x);
    return u;
}

bool has(const std::string &s, char c) { return s.find(c) != std::string::npos; }

}  // namespace

const_status_t parse_plan(const char *expression, const char *const *tree, int n_contractions,
                          const char *const *sparse_names, const int *const *mode_orders, int n_sparse,
                          const char *const *loop_orders, const const_extent_t *extents, int n_indices,
                          const_dtype_t dtype, PlanDesc &p) {
    if (!expression || !tree || n_contractions < 1 || n_contractions > 16 || !loop_orders || !extents ||
        n_indices < 1 || n_sparse < 0 || (n_sparse > 0 && (!sparse_names || !mode_orders)) ||
        (dtype != CONST_F32 && dtype != CONST_F64))
        return CONST_ERR_INVALID_ARG;
    p = PlanDesc();
    p.dtype = dtype;
    if (!parse_assignment(expression, p.result, p.inputs) || p.inputs.size() < 2) {
        p.error = "malformed expression";
        return CONST_ERR_INVALID_ARG;
    }
    for (int c = 0; c < n_contractions; ++c) {
        if (!tree[c] || !loop_orders[c]) return CONST_ERR_INVALID_ARG;
        Contraction k;
        std::vector<TensorRef> rhs;
        if (!parse_assignment(tree[c], k.out, rhs) || rhs.size() != 2) {
            p.error = "malformed contraction (need exactly two operands)";
            return CONST_ERR_INVALID_ARG;
        }
        k.lhs = rhs[0];
        k.rhs = rhs[1];
        k.loops = loop_orders[c];
        p.tree.push_back(k);
    }
    for (int e = 0; e < n_indices; ++e) {
        if (!std::isalpha((unsigned char)extents[e].index) || extents[e].extent < 1 ||
            p.extents.count(extents[e].index)) {
            p.error = "bad extent list";
            return CONST_ERR_INVALID_ARG;
        }
        p.extents[extents[e].index] = extents[e].extent;
    }
    for (int t = 0; t < n_sparse; ++t) {
        if (!sparse_names[t] || !mode_orders[t]) return CONST_ERR_INVALID_ARG;
        const TensorRef *ref = nullptr;
        for (const TensorRef &r : p.inputs) if (r.name == sparse_names[t]) ref = &r;
        if (!ref || p.mode_orders.count(ref->name)) {
            p.error = "sparse tensor name is not an input of the expression";
            return CONST_ERR_INVALID_ARG;
        }
        p.mode_orders[ref->name] = std::vector<int>(mode_orders[t], mode_orders[t] + ref->idx.size());
    }
    // every index needs an extent; input names are distinct
    std::set<std::string> names;
    for (const TensorRef &r : p.inputs) {
        if (!names.insert(r.name).second || r.name == p.result.name) {
            p.error = "tensor names of the expression must be distinct";
            return CONST_ERR_INVALID_ARG;
        }
        for (char x : r.idx) if (!p.extents.count(x)) { p.error = "index without extent"; return CONST_ERR_INVALID_ARG; }
    }
    for (char x : p.result.idx) if (!p.extents.count(x)) { p.error = "index without extent"; return CONST_ERR_INVALID_ARG; }
    return CONST_OK;
}

const_status_t check_plan(PlanDesc &p) {
    const int m = (int)p.tree.size();
    auto fail = [&](const char *why) { p.error = why; return CONST_ERR_ILLEGAL_SCHEDULE; };

    // Sec. 3.2.2: dp values of each CSF tensor form a permutation of its modes.
    for (auto &kv : p.mode_orders)
        if (!is_permutation(kv.second)) return fail("CSF mode order is not a permutation");

    // Sec. 3.2.1: the order of assignments is a topological order of the tree.  An operand is an
    // input of the network or the result of an earlier contraction; each input and each
    // intermediate feeds exactly one contraction.
    std::map<std::string, int> producer;           // tensor name -> contraction that writes it
    std::map<std::string, int> consumer;           // tensor name -> contraction that reads it
    std::map<std::string, std::string> ref_idx;    // tensor name -> indices of its (single) reference
    for (const TensorRef &r : p.inputs) ref_idx[r.name] = r.idx;
    for (int c = 0; c < m; ++c) {
        const Contraction &k = p.tree[c];
        for (const TensorRef *r : {&k.lhs, &k.rhs}) {
            bool is_input = false;
            for (const TensorRef &in : p.inputs) if (in.name == r->name) is_input = true;
            if (!is_input && !producer.count(r->name))
                return fail("operand is used before the contraction that produces it");
            if (consumer.count(r->name)) return fail("tensor is consumed by more than one contraction");
            if (ref_idx[r->name] != r->idx) return fail("tensor is referenced with different indices");
            consumer[r->name] = c;
        }
        if (producer.count(k.out.name) || ref_idx.count(k.out.name))
            return fail("result name of a contraction is already taken");
        producer[k.out.name] = c;
        ref_idx[k.out.name] = k.out.idx;
        for (char x : k.out.idx)
            if (!has(k.lhs.idx, x) && !has(k.rhs.idx, x)) return fail("result index does not occur in the operands");
        for (char x : index_union(k))
            if (!p.extents.count(x)) return fail("index without extent");
    }
    for (const TensorRef &in : p.inputs)
        if (!consumer.count(in.name)) return fail("an input of the expression is not used by the tree");
    for (int c = 0; c + 1 < m; ++c)
        if (!consumer.count(p.tree[c].out.name)) return fail("intermediate result is never consumed");
    const Contraction &root = p.tree[m - 1];
    if (root.out.name != p.result.name || root.out.idx != p.result.idx)
        return fail("last contraction does not produce the result of the expression");

    // The tree must compute the expression: an index summed by a contraction may not occur outside
    // the sub-tree of that contraction (otherwise distributivity does not apply, Sec. 2.1).
    std::vector<std::set<std::string>> leaves(m);
    for (int c = 0; c < m; ++c)
        for (const TensorRef *r : {&p.tree[c].lhs, &p.tree[c].rhs}) {
            if (producer.count(r->name)) {
                const auto &sub = leaves[producer[r->name]];
                leaves[c].insert(sub.begin(), sub.end());
            } else {
                leaves[c].insert(r->name);
            }
        }
    for (int c = 0; c < m; ++c) {
        const Contraction &k = p.tree[c];
        for (char x : index_union(k)) {
            if (has(k.out.idx, x)) continue;                       // external index of this contraction
            if (has(p.result.idx, x)) return fail("an index of the result is summed inside the tree");
            for (const TensorRef &in : p.inputs)
                if (!leaves[c].count(in.name) && has(in.idx, x))
                    return fail("an index is summed before all tensors that carry it have been multiplied");
        }
    }
    for (const TensorRef &in : p.inputs)
        for (char x : in.idx) {
            // an index carried by an input is either external or summed somewhere
            bool summed = false;
            for (int c = 0; c < m; ++c) {
                const Contraction &k = p.tree[c];
                if ((has(k.lhs.idx, x) || has(k.rhs.idx, x)) && !has(k.out.idx, x)) summed = true;
            }
            if (!summed && !has(p.result.idx, x)) return fail("index neither summed nor external");
        }

    // Sec. 3.2.3: lp values of each contraction form a permutation of its index set.
    for (int c = 0; c < m; ++c) {
        std::string u = index_union(p.tree[c]), l = p.tree[c].loops;
        std::string a = u, b = l;
        std::sort(a.begin(), a.end());
        std::sort(b.begin(), b.end());
        if (a != b) return fail("loop order is not a permutation of the contraction's indices");
    }

    // Sec. 3.2.4: (dp_j < dp_j') => (lp_k < lp_k') for every CSF operand.  Dense inputs and
    // intermediates kept in dense workspaces are exempt.
    for (int c = 0; c < m; ++c)
        for (const TensorRef *r : {&p.tree[c].lhs, &p.tree[c].rhs}) {
            auto it = p.mode_orders.find(r->name);
            if (it == p.mode_orders.end()) continue;
            size_t prev = 0;
            for (size_t l = 0; l < it->second.size(); ++l) {
                size_t at = p.tree[c].loops.find(r->idx[it->second[l]]);
                if (l > 0 && at < prev) return fail("loop order disagrees with the CSF level order of an operand");
                prev = at;
            }
        }

    // Sec. 3.2.5: producer / consumer / statements in between.  The loops removed from an
    // intermediate are the longest common loop prefix of every contraction from its producer to its
    // consumer, cut at the first loop that is not an index of the intermediate.
    p.fused_loops.assign(m, 0);
    p.reduced_order.assign(m, 0);
    for (int c = 0; c + 1 < m; ++c) {
        const Contraction &prod = p.tree[c];
        int q = consumer[prod.out.name];
        int f = 0;
        for (;; ++f) {
            if (f >= (int)prod.loops.size()) break;
            char x = prod.loops[f];
            if (!has(prod.out.idx, x)) break;
            bool same = true;
            for (int r = c + 1; r <= q; ++r)
                if (f >= (int)p.tree[r].loops.size() || p.tree[r].loops[f] != x) same = false;
            if (!same) break;
        }
        p.fused_loops[c] = f;
        p.reduced_order[c] = (int)prod.out.idx.size() - f;
    }
    return CONST_OK;
}

const_status_t match_plan(PlanDesc &p) {
    auto no = [&](const char *why) { p.error = why; p.family = Family::None; return CONST_ERR_UNSUPPORTED; };
    const int m = (int)p.tree.size();

    if (p.mode_orders.size() == 1) {
        // ---- chain family: one CSF tensor, one dense factor per non-root level ----
        const std::string xname = p.mode_orders.begin()->first;
        const std::vector<int> &mo = p.mode_orders.begin()->second;
        const int n = (int)mo.size();
        if (n != 3 && n != 4) return no("chain family needs a CSF tensor of order 3 or 4");
        if (m != n - 1 || (int)p.inputs.size() != n) return no("chain family needs one factor per non-root level");
        if (p.dtype != CONST_F32) return no("chain family computes in fp32");
        const TensorRef *X = nullptr;
        for (const TensorRef &r : p.inputs) if (r.name == xname) X = &r;
        std::string lev(n, ' ');
        for (int l = 0; l < n; ++l) lev[l] = X->idx[mo[l]];
        std::string cur = xname;                   // tensor carrying the not-yet-contracted levels
        std::vector<std::string> factors(n);       // factor of level l
        std::vector<char> rank_idx(n, 0);
        for (int c = 0; c < m; ++c) {
            const Contraction &k = p.tree[c];
            const int level = n - 1 - c;
            const TensorRef *fac = nullptr;
            if (k.lhs.name == cur) fac = &k.rhs;
            else if (k.rhs.name == cur) fac = &k.lhs;
            else return no("contractions do not form a leaf-to-root chain");

            if (p.mode_orders.count(fac->name) || fac->idx.size() != 2 || fac->idx[0] != lev[level])
                return no("factor must be a dense matrix indexed [level index, rank index]");
            if (has(k.out.idx, lev[level])) return no("each contraction must sum the innermost remaining level");
            factors[level] = fac->name;
            rank_idx[level] = fac->idx[1];
            cur = k.out.name;
        }
        bool all_same = true, all_distinct = true;
        for (int l = 1; l < n; ++l) {
            if (rank_idx[l] != rank_idx[1]) all_same = false;
            for (int l2 = 1; l2 < l; ++l2) if (rank_idx[l] == rank_idx[l2]) all_distinct = false;
        }
        std::string want_out(1, lev[0]);
        if (all_distinct) for (int l = 1; l < n; ++l) want_out.push_back(rank_idx[l]);
        else if (all_same) want_out.push_back(rank_idx[1]);
        else return no("rank indices must be all distinct (TTMc) or all equal (MTTKRP)");
        if (p.result.idx != want_out) return no("result must be indexed [root level, rank indices in level order]");
        for (int l = 1; l < n; ++l) {
            int64_t r = p.extents[rank_idx[l]];
            if (r != 8 && r != 16 && r != 32) return no("rank must be 8, 16 or 32");
            p.ranks.push_back((int)r);
        }
        // fusion depth: every intermediate keeps only what lies below the fused loops
        for (int c = 0; c + 1 < m; ++c) {
            const int level = n - 1 - c;           // level summed by contraction c
            if (p.fused_loops[c] != level) return no("loops above the contracted level must be fused");
            for (int f = 0; f < level; ++f)
                if (p.tree[c].loops[f] != lev[f]) return no("fused loops must follow the CSF levels");
        }
        if (all_distinct && n == 3) p.family = Family::Ttmc3;
        else if (all_distinct && n == 4) {
            if (p.ranks[0] != 8 || p.ranks[1] != 8 || p.ranks[2] != 8)
                return no("order-4 TTMc is implemented for rank 8");
            p.family = Family::Ttmc4;
        } else if (all_same && n == 3) p.family = Family::Mttkrp3;
        else return no("MTTKRP is implemented for order 3");
        p.sparse_name = xname;
        p.factor_names.assign(factors.begin() + 1, factors.end());
        return CONST_OK;
    }

    if (p.mode_orders.size() == 2 && m == 2 && p.inputs.size() == 3) {
        // ---- network family: T[i,k,l] = U[i,j,k] V[j,l];  Z[i,m] = T[i,k,l] W[k,l,m], fused over i ----
        if (p.dtype != CONST_F64) return no("network family computes in fp64");
        const Contraction &c0 = p.tree[0], &c1 = p.tree[1];
        const TensorRef *U = nullptr, *V = nullptr, *W = nullptr, *T = nullptr;
        for (const TensorRef *r : {&c0.lhs, &c0.rhs}) (p.mode_orders.count(r->name) ? U : V) = r;
        for (const TensorRef *r : {&c1.lhs, &c1.rhs}) (p.mode_orders.count(r->name) ? W : T) = r;
        if (!U || !V || !W || !T || T->name != c0.out.name) return no("not a sparse-dense-sparse network");
        if (U->idx.size() != 3 || W->idx.size() != 3 || V->idx.size() != 2 || T->idx.size() != 3 ||
            p.result.idx.size() != 2)
            return no("network family needs order-3 sparse tensors and a dense matrix");
        // gather-form schedule: U stored (i,k,j), W stored (l,m,k)
        const std::vector<int> &mu = p.mode_orders[U->name], &mw = p.mode_orders[W->name];
        char i = U->idx[mu[0]], k = U->idx[mu[1]], j = U->idx[mu[2]];
        char l = W->idx[mw[0]], mm = W->idx[mw[1]], wk = W->idx[mw[2]];
        if (wk != k) return no("W's leaf level must be the index it shares with U (U stored i,k,j; W stored l,m,k)");
        if (V->idx[0] != j || V->idx[1] != l) return no("V must be indexed [U's leaf index, W's root index]");
        std::string t = T->idx;
        std::sort(t.begin(), t.end());
        std::string want{i, k, l};
        std::sort(want.begin(), want.end());
        if (t != want) return no("intermediate must carry i, k, l");
        if (p.result.idx != std::string{i, mm}) return no("result must be indexed [i, m]");
        if (p.fused_loops[0] != 1 || c0.loops[0] != i) return no("the network must be fused over i only");
        p.family = Family::Network;
        p.sparse_name = U->name;
        p.sparse2_name = W->name;
        p.factor_names = {V->name};
        return CONST_OK;
    }
    return no("schedule matches no kernel family");
}

}  // namespace cb
