// Compiles a checked schedule into the programs of the generic executor (tree_exec.h).  Host only.
//
// The loop tree (loop_tree.cpp, built with sound fusion only) is flattened entry by entry.  For every
// forall the compiler decides how it iterates: a CSF operand of the assignments below it that carries the
// loop's index may drive the loop -- the loop then visits only the coordinates that operand stores -- if
// skipping the other coordinates cannot change anything that leaves the loop, i.e. if every assignment
// whose result is used outside the loop depends on that operand through the assignments inside it.
// Otherwise the loop runs over the dense range of its index.  Every other CSF operand carrying the index
// is looked up at each coordinate.
#include "tree_exec.h"

#include <algorithm>
#include <map>
#include <set>

#include "loop_tree.h"

namespace cb {
namespace tree {
namespace {

bool has(const std::string &s, char c) { return s.find(c) != std::string::npos; }

struct TensorInfo {
    enum Kind { SparseIn, DenseIn, SharedWs, PrivateWs, Result } kind = DenseIn;
    int slot = -1;                 // sparse slot, global slot, or producing contraction (private workspace)
    std::string addr_idx;          // indices that address it, in storage order (dense kinds)
    std::string levels;            // sparse: index of each CSF level
};

void count_statements(const LoopNode &n, std::vector<int> &out) {
    if (!n.is_loop) { out.push_back(n.contraction); return; }
    for (const LoopNode &c : n.body) count_statements(c, out);
}

struct Compiler {
    const PlanDesc &d;
    Compiled &out;
    LoopTree tree;
    std::vector<std::vector<const LoopNode *>> paths;
    std::map<char, int> idx_id;
    std::map<std::string, TensorInfo> tensors;
    std::map<std::string, int> producer, consumer;
    std::map<const LoopNode *, std::vector<int>> zero_at;     // forall node -> private workspaces (by producer) cleared in its body
    const char *why = nullptr;

    Compiler(const PlanDesc &desc, Compiled &o) : d(desc), out(o) {}

    bool fail(const char *w) { why = w; return false; }

    int64_t extent(char x) const { return d.extents.at(x); }

    bool setup() {
        const int m = (int)d.tree.size();
        if (m > kMaxStmts) return fail("too many contractions for the generic executor");
        tree = build_loop_tree(d.tree, true);
        paths = loop_paths(tree);
        for (const Contraction &c : d.tree)
            for (char x : c.loops)
                if (!idx_id.count(x)) { const int id = (int)idx_id.size(); idx_id[x] = id; }
        if ((int)idx_id.size() > kMaxIdx) return fail("too many iteration indices for the generic executor");
        out.index_names.assign(idx_id.size(), '?');
        for (auto &kv : idx_id) out.index_names[(size_t)kv.second] = kv.first;
        for (int c = 0; c < m; ++c) {
            producer[d.tree[c].out.name] = c;
            consumer[d.tree[c].lhs.name] = c;
            consumer[d.tree[c].rhs.name] = c;
        }
        // inputs
        for (const TensorRef &in : d.inputs) {
            TensorInfo t;
            auto mo = d.mode_orders.find(in.name);
            if (mo != d.mode_orders.end()) {
                if ((int)in.idx.size() > kMaxLevels || in.idx.size() < 2) return fail("CSF operands have order 2 to 4");
                if ((int)out.sparse_names.size() >= kMaxSparse) return fail("too many CSF operands for the generic executor");
                t.kind = TensorInfo::SparseIn;
                t.slot = (int)out.sparse_names.size();
                for (int mode : mo->second) t.levels.push_back(in.idx[(size_t)mode]);
                out.sparse_names.push_back(in.name);
            } else {
                t.kind = TensorInfo::DenseIn;
                t.addr_idx = in.idx;
                if (!add_global(t, in.name, 0, false)) return false;
            }
            tensors[in.name] = t;
        }
        // intermediates and the result
        for (int c = 0; c < m; ++c) {
            const Contraction &k = d.tree[c];
            TensorInfo t;
            if (c == m - 1) {
                t.kind = TensorInfo::Result;
                t.addr_idx = d.result.idx;
                if (!add_global(t, k.out.name, elems(t.addr_idx), false)) return false;
                out.result_slot = t.slot;
            } else if (tree.removed[c].empty()) {
                t.kind = TensorInfo::SharedWs;           // producer and consumer share no forall: lives in global memory
                t.addr_idx = k.out.idx;
                if (!add_global(t, "", elems(t.addr_idx), true)) return false;
            } else {
                t.kind = TensorInfo::PrivateWs;
                t.slot = c;
                t.addr_idx = tree.reduced[c].out.idx;
                zero_at[paths[c][tree.removed[c].size() - 1]].push_back(c);
            }
            if (elems(t.addr_idx) >= (1ll << 31) || (int)t.addr_idx.size() > kMaxRefIdx)
                return fail("a dense tensor of the schedule is too large for the generic executor");
            tensors[k.out.name] = t;
        }
        for (const TensorRef &in : d.inputs)
            if (tensors[in.name].kind == TensorInfo::DenseIn &&
                (elems(in.idx) >= (1ll << 31) || (int)in.idx.size() > kMaxRefIdx))
                return fail("a dense operand is too large for the generic executor");
        return true;
    }

    int64_t elems(const std::string &idx) const {
        int64_t n = 1;
        for (char x : idx) {
            n *= extent(x);
            if (n >= (1ll << 40)) return n;
        }
        return n;
    }

    bool add_global(TensorInfo &t, const std::string &name, int64_t n, bool workspace) {
        if ((int)out.global_names.size() >= kMaxDense) return fail("too many dense tensors for the generic executor");
        t.slot = (int)out.global_names.size();
        out.global_names.push_back(name);
        out.global_elems.push_back(n);
        out.global_is_workspace.push_back(workspace);
        return true;
    }

    // ---- one reference of an assignment ----
    bool make_ref(const TensorRef &r, const Program &p, Ref &ref) {
        const TensorInfo &t = tensors.at(r.name);
        ref = Ref{};
        if (t.kind == TensorInfo::SparseIn) {
            ref.kind = kRefSparse;
            ref.slot = (int8_t)t.slot;
            return true;
        }
        ref.kind = t.kind == TensorInfo::PrivateWs ? kRefPrivate : kRefGlobal;
        ref.slot = (int8_t)t.slot;
        ref.n = (int8_t)t.addr_idx.size();
        int64_t stride = 1;
        for (int k = ref.n - 1; k >= 0; --k) {
            ref.idx[k] = (int8_t)idx_id.at(t.addr_idx[(size_t)k]);
            ref.stride[k] = (int32_t)stride;
            stride *= extent(t.addr_idx[(size_t)k]);
        }
        (void)p;
        return true;
    }

    // ---- how one forall iterates ----
    // stmts: the assignments below the forall; bound: the indices of the foralls around it
    bool make_loop(const LoopNode &node, const std::vector<int> &stmts, const std::string &bound, Loop &loop) {
        loop = Loop{};
        loop.index = (int8_t)idx_id.at(node.index);
        loop.driver = -1;
        loop.extent = (int32_t)std::min<int64_t>(extent(node.index), 0x7fffffff);
        if (extent(node.index) > 0x7fffffff) return fail("index extent too large");
        const std::set<int> inside(stmts.begin(), stmts.end());
        // assignments whose result leaves the loop
        std::vector<int> exits;
        for (int c : stmts) {
            auto q = consumer.find(d.tree[c].out.name);
            if (q == consumer.end() || !inside.count(q->second)) exits.push_back(c);
        }
        // does assignment e depend on assignment s through assignments inside the loop?
        auto depends = [&](int e, int s) {
            std::vector<int> todo{e};
            while (!todo.empty()) {
                const int c = todo.back();
                todo.pop_back();
                if (c == s) return true;
                for (const TensorRef *r : {&d.tree[c].lhs, &d.tree[c].rhs}) {
                    auto p = producer.find(r->name);
                    if (p != producer.end() && inside.count(p->second)) todo.push_back(p->second);
                }
            }
            return false;
        };
        struct Cand { int slot, level; bool valid; };
        std::vector<Cand> cands;
        for (int c : stmts)
            for (const TensorRef *r : {&d.tree[c].lhs, &d.tree[c].rhs}) {
                const TensorInfo &t = tensors.at(r->name);
                if (t.kind != TensorInfo::SparseIn || !has(t.levels, node.index)) continue;
                const int level = (int)t.levels.find(node.index);
                for (int l = 0; l < level; ++l)
                    if (!has(bound, t.levels[(size_t)l])) return fail("a loop order does not follow the CSF level order of an operand");
                bool valid = true;
                for (int e : exits) valid = valid && depends(e, c);
                cands.push_back(Cand{t.slot, level, valid});
            }
        int best = -1;
        for (size_t k = 0; k < cands.size(); ++k)
            if (cands[k].valid && (best < 0 || cands[k].level > cands[(size_t)best].level)) best = (int)k;
        for (size_t k = 0; k < cands.size(); ++k) {
            if ((int)k == best) {
                loop.driver = (int8_t)cands[k].slot;
                loop.level = (int8_t)cands[k].level;
            } else {
                if (loop.n_follow >= kMaxFollow) return fail("too many CSF operands share one loop index");
                loop.follow[loop.n_follow] = (int8_t)cands[k].slot;
                loop.flevel[loop.n_follow] = (int8_t)cands[k].level;
                ++loop.n_follow;
            }
        }
        return true;
    }

    // ---- flattening ----
    struct Emit {
        Program p{};
        int n_loops = 0, n_stmts = 0;
        std::map<int, int> ws_id;         // producing contraction -> workspace id of this program
        std::vector<std::string> stmt_text, ws_text;
    };

    static std::string show(const TensorRef &r) {
        std::string t = r.name + "(";
        for (size_t i = 0; i < r.idx.size(); ++i) { if (i) t += ", "; t.push_back(r.idx[i]); }
        return t + ")";
    }

    bool new_loop(Emit &e, const LoopNode &node, const std::vector<int> &stmts, const std::string &bound, int &id) {
        if (e.n_loops >= kMaxLoops) return fail("too many loops for the generic executor");
        id = e.n_loops++;
        return make_loop(node, stmts, bound, e.p.loops[id]);
    }

    bool push(Emit &e, Op op, int arg, int &at) {
        if (e.p.n_instr >= kMaxInstr) return fail("schedule too long for the generic executor");
        at = e.p.n_instr++;
        e.p.instr[at] = Instr{(int8_t)op, (int8_t)arg, 0};
        return true;
    }

    bool emit_zeros(Emit &e, const LoopNode *owner) {
        auto z = zero_at.find(owner);
        if (z == zero_at.end()) return true;
        for (int c : z->second) {
            int at;
            if (!push(e, kOpZero, e.ws_id.at(c), at)) return false;
        }
        return true;
    }

    // an assignment with the chain of private foralls `chain` around it (outermost first)
    bool emit_statement(Emit &e, int c, const std::vector<const LoopNode *> &chain, std::string bound) {
        if (e.n_stmts >= kMaxStmts) return fail("too many assignments for the generic executor");
        Stmt &s = e.p.stmts[e.n_stmts];
        s = Stmt{};
        if ((int)chain.size() > kMaxPriv) return fail("loop nest too deep for the generic executor");
        for (const LoopNode *n : chain) {
            int id;
            if (!new_loop(e, *n, {c}, bound, id)) return false;
            s.priv[s.n_priv++] = (int8_t)id;
            bound.push_back(n->index);
        }
        if (s.n_priv >= 2) {
            const Loop &inner = e.p.loops[s.priv[s.n_priv - 1]], &outer = e.p.loops[s.priv[s.n_priv - 2]];
            s.fuse_tail = inner.driver < 0 && inner.n_follow == 0 && outer.n_follow == 0 &&
                          (int64_t)inner.extent * outer.extent < (1ll << 31);
        }
        const Contraction &k = d.tree[c];
        if (!make_ref(k.out, e.p, s.out) || !make_ref(k.lhs, e.p, s.lhs) || !make_ref(k.rhs, e.p, s.rhs)) return false;
        for (const Ref *r : {&s.lhs, &s.rhs})
            if (r->kind == kRefSparse) s.sparse[s.n_sparse++] = r->slot;
        if (s.out.kind == kRefPrivate) s.out.slot = (int8_t)e.ws_id.at(s.out.slot);
        if (s.lhs.kind == kRefPrivate) s.lhs.slot = (int8_t)e.ws_id.at(s.lhs.slot);
        if (s.rhs.kind == kRefPrivate) s.rhs.slot = (int8_t)e.ws_id.at(s.rhs.slot);
        if (s.n_priv >= 1) {
            const Loop &LB = e.p.loops[s.priv[s.n_priv - 1]];
            const Loop *LA = s.fuse_tail ? &e.p.loops[s.priv[s.n_priv - 2]] : nullptr;
            s.fast = LB.n_follow == 0 && (!LA || LA->n_follow == 0);
            const TensorRef *names[3] = {&k.out, &k.lhs, &k.rhs};
            const Ref *refs[3] = {&s.out, &s.lhs, &s.rhs};
            for (int r = 0; r < 3; ++r) {
                const Ref &ref = *refs[r];
                if (ref.kind == kRefSparse) {
                    const int leaf = (int)tensors.at(names[r]->name).levels.size() - 1;
                    s.pB[r] = LB.driver == ref.slot && LB.level == leaf;
                    s.pA[r] = LA && LA->driver == ref.slot && LA->level == leaf;
                } else {
                    for (int x = 0; x < ref.n; ++x) {
                        if (ref.idx[x] == LB.index) s.sB[r] = ref.stride[x];
                        if (LA && ref.idx[x] == LA->index) s.sA[r] = ref.stride[x];
                    }
                }
            }
        }
        const Contraction &rk = tree.reduced[c];
        e.stmt_text.push_back(show(rk.out) + " += " + show(rk.lhs) + " * " + show(rk.rhs));
        int at;
        return push(e, kOpStmt, e.n_stmts++, at);
    }

    bool emit_node(Emit &e, const LoopNode &n, const std::string &bound) {
        std::vector<int> stmts;
        count_statements(n, stmts);
        if (stmts.size() == 1) {
            std::vector<const LoopNode *> chain;
            const LoopNode *cur = &n;
            while (cur->is_loop) { chain.push_back(cur); cur = &cur->body[0]; }
            return emit_statement(e, stmts[0], chain, bound);
        }
        int id, begin, end;
        if (!new_loop(e, n, stmts, bound, id) || !push(e, kOpLoopBegin, id, begin)) return false;
        if (!emit_zeros(e, &n)) return false;
        for (const LoopNode &c : n.body)
            if (!emit_node(e, c, bound + n.index)) return false;
        if (!push(e, kOpLoopEnd, id, end)) return false;
        e.p.instr[begin].jump = (int16_t)(end + 1);     // an empty range skips the body
        e.p.instr[end].jump = (int16_t)(begin + 1);     // the next iteration re-enters behind the begin
        return true;
    }

    bool emit_root(const LoopNode &root, int &driver, int64_t &root_extent) {
        Emit e;
        std::vector<int> stmts;
        count_statements(root, stmts);
        // private workspaces of this entry
        for (int c : stmts)
            if (tensors.at(d.tree[c].out.name).kind == TensorInfo::PrivateWs) {
                const int id = (int)e.ws_id.size();
                e.ws_id[c] = id;
                const int64_t n = elems(tree.reduced[c].out.idx);
                e.p.ws[id] = Workspace{e.p.block_scratch, n};
                e.ws_text.push_back(show(tree.reduced[c].out));
                e.p.block_scratch += (n + 1) / 2 * 2;           // keeps 16-byte alignment for fp64
            }
        driver = -1;
        root_extent = 1;
        e.p.root_loop = -1;
        e.p.root_loop2 = -1;
        if (!root.is_loop) {
            if (!emit_statement(e, root.contraction, {}, "")) return false;
        } else if (stmts.size() == 1) {
            // a single assignment: its outermost loop goes to the blocks, the rest stays private
            std::vector<const LoopNode *> chain;
            const LoopNode *cur = &root;
            while (cur->is_loop) { chain.push_back(cur); cur = &cur->body[0]; }
            int id;
            if (!new_loop(e, root, stmts, "", id)) return false;
            e.p.root_loop = id;
            chain.erase(chain.begin());
            if (!emit_statement(e, stmts[0], chain, std::string(1, root.index))) return false;
        } else {
            int id;
            if (!new_loop(e, root, stmts, "", id)) return false;
            e.p.root_loop = id;
            // Two fused loops at once: when the body of the outermost loop is nothing but the next fused loop, and
            // both walk consecutive levels of the same CSF operand, a block takes one level-1 node of that operand
            // (a pair of coordinates) instead of a whole level-0 node: far more blocks, far more evenly loaded.
            const LoopNode *inner = root.body.size() == 1 && root.body[0].is_loop ? &root.body[0] : nullptr;
            std::vector<int> inner_stmts;
            if (inner) count_statements(*inner, inner_stmts);
            bool flattened = false;
            if (inner && inner_stmts.size() >= 2 && !zero_at.count(&root) && e.p.loops[id].driver >= 0) {
                int id2;
                if (!new_loop(e, *inner, inner_stmts, std::string(1, root.index), id2)) return false;
                if (e.p.loops[id2].driver == e.p.loops[id].driver && e.p.loops[id2].level == 1) {
                    e.p.root_loop2 = id2;
                    if (!emit_zeros(e, inner)) return false;
                    for (const LoopNode &c : inner->body)
                        if (!emit_node(e, c, std::string(1, root.index) + inner->index)) return false;
                    flattened = true;
                } else {
                    --e.n_loops;                                  // not the same operand: the inner loop stays a uniform loop
                }
            }
            if (!flattened) {
                if (!emit_zeros(e, &root)) return false;
                for (const LoopNode &c : root.body)
                    if (!emit_node(e, c, std::string(1, root.index))) return false;
            }
        }
        if (e.p.root_loop >= 0) {
            driver = e.p.loops[e.p.root_loop].driver;
            root_extent = extent(root.index);
        }
        out.programs.push_back(e.p);
        out.root_flattened.push_back(e.p.root_loop2 >= 0);
        out.stmt_text.push_back(e.stmt_text);
        out.ws_text.push_back(e.ws_text);
        return true;
    }

    bool run() {
        if (!setup()) return false;
        for (const LoopNode &root : tree.roots) {
            int driver;
            int64_t ext;
            if (!emit_root(root, driver, ext)) return false;
            out.root_driver.push_back(driver);
            out.root_extent.push_back(ext);
        }
        return true;
    }
};

}  // namespace

std::string describe(const Compiled &c) {
    std::string text;
    auto loop_text = [&](const Loop &L) {
        std::string t(1, c.index_names[(size_t)L.index]);
        if (L.driver >= 0) t += ": walks " + c.sparse_names[(size_t)L.driver] + " level " + std::to_string(L.level);
        else t += ": dense range 0.." + std::to_string(L.extent);
        for (int f = 0; f < L.n_follow; ++f)
            t += std::string(f ? ", " : "; locates ") + c.sparse_names[(size_t)L.follow[f]] + " level " + std::to_string(L.flevel[f]);
        return t;
    };
    for (size_t r = 0; r < c.programs.size(); ++r) {
        const Program &p = c.programs[r];
        text += "entry " + std::to_string(r) + ": ";
        text += p.root_loop >= 0 ? "blocks over " + loop_text(p.loops[p.root_loop]) : std::string("one block");
        if (p.root_loop2 >= 0) text += " | and over " + loop_text(p.loops[p.root_loop2]);
        text += "\n";
        int depth = 1;
        for (int pc = 0; pc < p.n_instr; ++pc) {
            const Instr in = p.instr[pc];
            if (in.op == kOpLoopEnd) { --depth; continue; }
            text += std::string(2 * (size_t)depth, ' ');
            if (in.op == kOpLoopBegin) {
                text += "loop " + loop_text(p.loops[in.arg]) + "\n";
                ++depth;
            } else if (in.op == kOpZero) {
                text += "zero " + c.ws_text[r][(size_t)in.arg] + " (" + std::to_string(p.ws[in.arg].size) + " elements per iteration in flight)\n";
            } else {
                const Stmt &st = p.stmts[in.arg];
                text += c.stmt_text[r][(size_t)in.arg];
                for (int k = 0; k < st.n_priv; ++k)
                    text += std::string(k ? ", " : "  [private loops: ") + loop_text(p.loops[st.priv[k]]);
                text += st.n_priv ? (st.fuse_tail ? "; last two dealt out as one]\n" : "]\n") : "\n";
            }
        }
    }
    return text;
}

bool compile(const PlanDesc &desc, Compiled &out) {
    out = Compiled();
    Compiler c(desc, out);
    if (!c.run()) {
        out.error = c.why ? c.why : "schedule cannot be compiled for the generic executor";
        out.programs.clear();
        return false;
    }
    return true;
}

}  // namespace tree
}  // namespace cb
