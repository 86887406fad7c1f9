// Loop tree of a schedule (Sec. 4.2): the sequence of <assignment, loop permutation> pairs arranged as
// nested forall loops whose bodies are lists of loops and assignments in execution order.  A body with
// several entries is a producer / consumer chain: the last entry consumes what the entries before it
// produce (the where(C, P) construct of Sec. 4.1).  The tree is what Algorithm 1 prints; here it is a data
// structure first, printed as concrete index notation by `print_cin` and walked by the generic executor.
#pragma once
#include <string>
#include <vector>

#include "plan.h"

namespace cb {

struct LoopNode {
    bool is_loop = false;
    char index = 0;                    // is_loop: the forall index
    int contraction = -1;              // !is_loop: position of the assignment in the sequence
    std::vector<LoopNode> body;        // is_loop: entries in execution order
};

struct LoopTree {
    std::vector<LoopNode> roots;       // top-level entries in execution order
    // The assignments as they stand inside the tree: an intermediate has lost every index whose forall
    // encloses both its producer and its consumer (it is a dense workspace over the remaining indices).
    std::vector<Contraction> reduced;
    // per contraction: the indices removed from its result by fusion, outermost first
    std::vector<std::string> removed;
};

// seq: the assignments with their loop permutations (Contraction::loops), references in the order they are
// to be printed.  only_sound_fusion = false groups consecutive pairs whenever their leading loops agree,
// as Algorithm 1 does; true additionally refuses to put a producer and its consumer under a common forall
// whose index the intermediate does not carry (the consumer would read partial sums), which is what the
// executor needs.
LoopTree build_loop_tree(const std::vector<Contraction> &seq, bool only_sound_fusion);

std::string print_cin(const LoopTree &t);

// per assignment: the forall nodes around it, outermost first (pointers into `t`)
std::vector<std::vector<const LoopNode *>> loop_paths(const LoopTree &t);

}  // namespace cb
