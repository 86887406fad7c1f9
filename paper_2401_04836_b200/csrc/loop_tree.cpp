// Loop tree of a schedule and its concrete index notation (Sec. 4.1, 4.2; behaviour of Algorithm 1).
//
// Construction.  The sequence is cut into maximal runs of consecutive pairs that share their leading loop
// index; a run becomes one forall node whose body is built the same way from the run with that loop taken
// off, and a pair with no loops left becomes an assignment.  Afterwards every intermediate is reduced: the
// foralls that enclose both its producer and its consumers are exactly the common prefix of their paths
// from the root, and their indices are dropped from every reference to it.  Printing a list of entries
// nests them as where(last, where(..., first)), which is what Algorithm 1 emits for the same input.
#include "loop_tree.h"

#include <algorithm>

namespace cb {
namespace {

struct Item {
    int c;                  // position in the sequence
    std::string loops;      // loops not yet turned into foralls, outermost first
};

bool reads(const Contraction &k, const std::string &name) { return k.lhs.name == name || k.rhs.name == name; }

// May `next` join a run under forall(x)?  Not if it consumes the result of a member of the run that does
// not carry x: inside the loop it would see that result before the sum over x is complete.
bool sound_to_join(const std::vector<Item> &run, const Item &next, char x, const std::vector<Contraction> &seq) {
    for (const Item &p : run)
        if (reads(seq[next.c], seq[p.c].out.name) && seq[p.c].out.idx.find(x) == std::string::npos) return false;
    return true;
}

std::vector<LoopNode> arrange(const std::vector<Item> &items, const std::vector<Contraction> &seq, bool sound) {
    std::vector<LoopNode> out;
    size_t k = 0;
    while (k < items.size()) {
        LoopNode node;
        if (items[k].loops.empty()) {
            node.contraction = items[k].c;
            out.push_back(node);
            ++k;
            continue;
        }
        const char x = items[k].loops[0];
        std::vector<Item> run;
        while (k < items.size() && !items[k].loops.empty() && items[k].loops[0] == x &&
               (run.empty() || !sound || sound_to_join(run, items[k], x, seq))) {
            run.push_back(Item{items[k].c, items[k].loops.substr(1)});
            ++k;
        }
        node.is_loop = true;
        node.index = x;
        node.body = arrange(run, seq, sound);
        out.push_back(node);
    }
    return out;
}

// path[c] = the forall nodes around assignment c, outermost first
void collect_paths(const std::vector<LoopNode> &list, std::vector<const LoopNode *> &stack,
                   std::vector<std::vector<const LoopNode *>> &path) {
    for (const LoopNode &n : list) {
        if (!n.is_loop) {
            path[n.contraction] = stack;
            continue;
        }
        stack.push_back(&n);
        collect_paths(n.body, stack, path);
        stack.pop_back();
    }
}

void drop(TensorRef &r, char x) { r.idx.erase(std::remove(r.idx.begin(), r.idx.end(), x), r.idx.end()); }

std::string show_ref(const TensorRef &r) {
    std::string s = r.name + "(";
    for (size_t i = 0; i < r.idx.size(); ++i) {
        if (i) s += ", ";
        s.push_back(r.idx[i]);
    }
    return s + ")";
}

std::string show_list(const std::vector<LoopNode> &list, size_t count, const LoopTree &t);

std::string show_node(const LoopNode &n, const LoopTree &t) {
    if (!n.is_loop) {
        const Contraction &c = t.reduced[n.contraction];
        return show_ref(c.out) + " = " + show_ref(c.lhs) + " * " + show_ref(c.rhs);
    }
    return std::string("forall(") + n.index + ", " + show_list(n.body, n.body.size(), t) + ")";
}

// the first `count` entries of a body: the last of them consumes, the ones before it produce
std::string show_list(const std::vector<LoopNode> &list, size_t count, const LoopTree &t) {
    if (count == 0) return "";
    if (count == 1) return show_node(list[0], t);
    return "where(" + show_node(list[count - 1], t) + ", " + show_list(list, count - 1, t) + ")";
}

}  // namespace

LoopTree build_loop_tree(const std::vector<Contraction> &seq, bool only_sound_fusion) {
    LoopTree t;
    std::vector<Item> items;
    for (size_t c = 0; c < seq.size(); ++c) items.push_back(Item{(int)c, seq[c].loops});
    t.roots = arrange(items, seq, only_sound_fusion);
    t.reduced = seq;
    t.removed.assign(seq.size(), "");
    std::vector<std::vector<const LoopNode *>> path(seq.size());
    std::vector<const LoopNode *> stack;
    collect_paths(t.roots, stack, path);
    for (size_t p = 0; p < seq.size(); ++p) {
        const std::string name = seq[p].out.name;
        size_t shared = path[p].size();
        bool consumed = false;
        for (size_t q = 0; q < seq.size(); ++q) {
            if (q == p || !reads(seq[q], name)) continue;
            consumed = true;
            size_t d = 0;
            while (d < shared && d < path[q].size() && path[q][d] == path[p][d]) ++d;
            shared = d;
        }
        if (!consumed) continue;
        for (size_t d = 0; d < shared; ++d) {
            const char x = path[p][d]->index;
            if (seq[p].out.idx.find(x) == std::string::npos) continue;
            t.removed[p].push_back(x);
            for (Contraction &k : t.reduced) {
                if (k.out.name == name) drop(k.out, x);
                if (k.lhs.name == name) drop(k.lhs, x);
                if (k.rhs.name == name) drop(k.rhs, x);
            }
        }
    }
    return t;
}

std::string print_cin(const LoopTree &t) { return show_list(t.roots, t.roots.size(), t); }

std::vector<std::vector<const LoopNode *>> loop_paths(const LoopTree &t) {
    std::vector<std::vector<const LoopNode *>> path(t.reduced.size());
    std::vector<const LoopNode *> stack;
    collect_paths(t.roots, stack, path);
    return path;
}

// References are written as the schedule stores them: a sparse input by its CSF mode order (dp), an
// intermediate and the result by the loop order of the contraction that produces them, which the
// consistency constraint of Sec. 3.2.4 makes agree with every permutation that reads a CSF tensor.
std::string schedule_cin(const PlanDesc &p) {
    std::map<std::string, std::string> layout;      // tensor name -> index order of its references
    for (const TensorRef &in : p.inputs) {
        auto mo = p.mode_orders.find(in.name);
        if (mo == p.mode_orders.end() || mo->second.size() != in.idx.size()) continue;   // kept as written
        std::string order;
        for (int mode : mo->second) order.push_back(in.idx[(size_t)mode]);
        layout[in.name] = order;
    }
    for (const Contraction &c : p.tree) {
        bool all_loops = true;
        for (char x : c.out.idx) all_loops = all_loops && c.loops.find(x) != std::string::npos;
        if (!all_loops) continue;                   // a sequence whose fused loops are already gone: kept as written
        std::string order = c.out.idx;
        std::stable_sort(order.begin(), order.end(),
                         [&](char x, char y) { return c.loops.find(x) < c.loops.find(y); });
        layout[c.out.name] = order;
    }
    auto relayout = [&](TensorRef r) {
        auto it = layout.find(r.name);
        if (it == layout.end()) return r;
        std::string idx;
        for (char c : it->second) if (r.idx.find(c) != std::string::npos) idx.push_back(c);
        if (idx.size() == r.idx.size()) r.idx = idx;
        return r;
    };
    std::vector<Contraction> seq;
    for (const Contraction &c : p.tree) {
        Contraction q;
        q.out = relayout(c.out);
        q.lhs = relayout(c.lhs);
        q.rhs = relayout(c.rhs);
        q.loops = c.loops;
        seq.push_back(q);
    }
    return print_cin(build_loop_tree(seq, false));
}

}  // namespace cb
