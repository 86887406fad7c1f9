// Concrete index notation of a schedule (Sec. 4.2, Algorithm 1): the sequence of <assignment, loop
// permutation> pairs becomes a nest of forall(index, ...) and where(consumer, producer) constructs.
// Host only.  The recursion follows the algorithm's two stages: group the pairs of a level by their
// outermost loop index, then emit either the single assignment, a forall around the group of a single
// index (after `remove`), or a where whose consumer is the group of the last element and whose producer
// is everything before it.
#include "plan.h"

#include <algorithm>

namespace cb {
namespace {

struct Pair {
    Contraction a;      // the assignment; a.loops is the permutation pi, outermost first
};

std::string show_ref(const TensorRef &r) {
    std::string s = r.name + "(";
    for (size_t i = 0; i < r.idx.size(); ++i) {
        if (i) s += ", ";
        s.push_back(r.idx[i]);
    }
    return s + ")";
}

std::string show_assignment(const Contraction &c) {
    return show_ref(c.out) + " = " + show_ref(c.lhs) + " * " + show_ref(c.rhs);
}

void drop_index(TensorRef &r, char i) { r.idx.erase(std::remove(r.idx.begin(), r.idx.end(), i), r.idx.end()); }

// The helper the paper describes in prose: strip the loop index i from the front of every permutation,
// and from every reference to an intermediate whose producer and consumer are both among `pairs`
// (both then sit inside forall(i, ...), so the intermediate loses that mode).
std::vector<Pair> remove_index(char i, std::vector<Pair> pairs) {
    for (Pair &p : pairs)
        if (!p.a.loops.empty() && p.a.loops[0] == i) p.a.loops.erase(0, 1);
    for (size_t prod = 0; prod < pairs.size(); ++prod) {
        const std::string name = pairs[prod].a.out.name;
        bool consumed_here = false;
        for (size_t c = 0; c < pairs.size(); ++c)
            if (c != prod && (pairs[c].a.lhs.name == name || pairs[c].a.rhs.name == name)) consumed_here = true;
        if (!consumed_here) continue;
        for (Pair &p : pairs) {
            if (p.a.out.name == name) drop_index(p.a.out, i);
            if (p.a.lhs.name == name) drop_index(p.a.lhs, i);
            if (p.a.rhs.name == name) drop_index(p.a.rhs, i);
        }
    }
    return pairs;
}

std::string generate(const std::vector<Pair> &S) {
    // stage 1: the list L of loop indices and assignments of this level; groups[e] = pairs of element e
    struct Element { bool is_index; char index; };
    std::vector<Element> L;
    std::vector<std::vector<Pair>> groups;
    for (const Pair &p : S) {
        if (p.a.loops.empty()) {
            L.push_back({false, 0});
            groups.push_back({p});
        } else {
            const char i = p.a.loops[0];
            if (L.empty() || !L.back().is_index || L.back().index != i) {
                L.push_back({true, i});
                groups.emplace_back();
            }
            groups.back().push_back(p);
        }
    }
    if (L.empty()) return "";
    // stage 2
    if (L.size() == 1) {
        if (!L[0].is_index) return show_assignment(groups[0][0].a);
        return std::string("forall(") + L[0].index + ", " + generate(remove_index(L[0].index, groups[0])) + ")";
    }
    const std::vector<Pair> &consumer = groups.back();
    std::vector<Pair> producer(S.begin(), S.end() - (std::ptrdiff_t)consumer.size());
    return "where(" + generate(consumer) + ", " + generate(producer) + ")";
}

}  // namespace

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
    std::vector<Pair> S;
    for (const Contraction &c : p.tree) {
        Pair q;
        q.a.out = relayout(c.out);
        q.a.lhs = relayout(c.lhs);
        q.a.rhs = relayout(c.rhs);
        q.a.loops = c.loops;
        S.push_back(q);
    }
    return generate(S);
}

}  // namespace cb
