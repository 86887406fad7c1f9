// Generic executor for loop trees (any legal schedule): the compiled form of a schedule that the
// interpreter kernel of tree_kernel.cu walks.  One Program per top-level entry of the loop tree.
//
// Execution model.  The outermost forall of an entry is spread over thread blocks.  Below it, a forall
// whose body holds several assignments ("uniform loop") is run by all threads of the block in lockstep,
// with a block barrier after every entry of its body; a forall chain that leads to a single assignment
// ("private loops") is run in parallel: its first loop is dealt to the warps, its second to the lanes,
// deeper ones run sequentially in each thread.  A loop walks the children of one CSF operand (its driver)
// when one qualifies, otherwise the dense range of its index; the other CSF operands that carry the index
// are located by binary search and an assignment is skipped where one of its operands has no such node.
// Intermediates are dense workspaces over the indices fusion left them: private to a block when producer
// and consumer share a forall (cleared at every iteration of the innermost shared one), global otherwise.
// All accumulation is by atomic adds, so results can differ in the last bits from run to run.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

#include "plan.h"

namespace cb {
namespace tree {

constexpr int kMaxIdx = 16, kMaxLoops = 24, kMaxStmts = 12, kMaxSparse = 6, kMaxDense = 20, kMaxInstr = 96;
constexpr int kMaxRefIdx = 6, kMaxPriv = 6, kMaxFollow = 3, kMaxLevels = 4;
constexpr int kThreads = 256;

enum RefKind : int8_t { kRefSparse = 0, kRefGlobal = 1, kRefPrivate = 2 };

struct Ref {                       // one tensor reference of an assignment
    int8_t kind;                   // RefKind
    int8_t slot;                   // sparse slot, global pointer slot, or private workspace id
    int8_t n;                      // indices that address it (global / private)
    int8_t idx[kMaxRefIdx];        // index ids
    int32_t stride[kMaxRefIdx];    // elements
};

struct Loop {
    int8_t index;                  // index id
    int8_t driver;                 // sparse slot whose level `level` the loop walks; -1: dense range [0, extent)
    int8_t level;
    int8_t n_follow;
    int8_t follow[kMaxFollow];     // sparse slots located at the loop's coordinate ...
    int8_t flevel[kMaxFollow];     // ... and the level of each that carries this index
    int32_t extent;
};

struct Stmt {
    int8_t n_priv;                 // private loops, outermost first
    int8_t priv[kMaxPriv];         // loop ids
    int8_t n_sparse;
    int8_t sparse[2];              // sparse slots it reads
    int8_t fuse_tail;              // the innermost private loop is a plain dense range and the one around it locates no
                                   // operand: the pair is dealt to the threads as one loop over their combined range
    Ref out, lhs, rhs;
    // Strength reduction of the innermost dealt loop (the last private loop, or the last two when fuse_tail):
    // when neither of them locates an operand (`fast`), the element a reference touches there is
    //   base + coordinate_A * sA + coordinate_B * sB + position_A * pA + position_B * pB
    // with A the outer and B the inner of the two (A unused without fuse_tail), `base` taken once per entry into
    // the loop, coordinate = the index value, position = the place in the driving operand's level.  Dense
    // references use sA / sB (their strides for the two indices), a sparse reference whose leaf level one of the
    // two loops walks uses pA / pB = 1, any other sparse reference is a constant of the loop.
    int8_t fast;
    int32_t sA[3], sB[3];          // out, lhs, rhs
    int8_t pA[3], pB[3];
};

enum Op : int8_t { kOpLoopBegin = 0, kOpLoopEnd = 1, kOpZero = 2, kOpStmt = 3 };
struct Instr { int8_t op; int8_t arg; int16_t jump; };

struct Workspace { int64_t offset, size; };      // block-private: elements, offset inside the block's scratch

struct Program {
    int32_t n_instr;
    int32_t root_loop;             // loop spread over the blocks, -1: the entry is a bare assignment
    int32_t root_loop2;            // >= 0: the loop below it, walking level 1 of the same operand, is spread over the
                                   // blocks together with it: a block takes one level-1 node (two fused loops at once)
    int64_t block_scratch;         // elements of private workspace per block
    Instr instr[kMaxInstr];
    Loop loops[kMaxLoops];
    Stmt stmts[kMaxStmts];
    Workspace ws[kMaxStmts];
};

struct SparsePtrs {
    const int32_t *pos[kMaxLevels];
    const int32_t *crd[kMaxLevels];
    const void *vals;
    int32_t n0, order;
};

struct Bindings {
    SparsePtrs sp[kMaxSparse];
    void *global[kMaxDense];       // dense inputs, the result, global workspaces
    void *scratch;                 // private workspaces: block b owns [b * block_scratch, (b + 1) * block_scratch);
                                   // NULL: they fit in the block's shared memory and live there
};

// What const_execute needs besides the programs.
struct Compiled {
    std::vector<Program> programs;
    std::vector<std::string> sparse_names;                 // slot -> input name
    std::vector<std::string> global_names;                 // slot -> input name, result name, or "" for a workspace
    std::vector<int64_t> global_elems;                     // slot -> elements (workspaces and the result; 0 for inputs)
    std::vector<bool> global_is_workspace;
    int result_slot = -1;
    std::vector<int> root_driver;                          // per program: sparse slot driving the root loop or -1
    std::vector<bool> root_flattened;                      // per program: blocks take level-1 nodes of that operand
    std::vector<int64_t> root_extent;                      // per program: extent of the root index (dense root loop)
    std::string index_names;                               // index id -> letter
    std::vector<std::vector<std::string>> stmt_text;       // per program, per statement: the assignment as it stands in the tree
    std::vector<std::vector<std::string>> ws_text;         // per program, per private workspace: its reduced reference
    std::string error;
};

// Human-readable listing of the compiled programs: how every loop iterates and what each entry does.
std::string describe(const Compiled &c);

// Compiles a parsed and checked schedule.  False (with `error` set) when it exceeds the fixed capacities.
bool compile(const PlanDesc &desc, Compiled &out);

}  // namespace tree
}  // namespace cb
