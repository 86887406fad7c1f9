// Host-side schedule descriptor: parsing, legality check (Sec. 3.2) and kernel-family matching.
#pragma once
#include <cstdint>
#include <map>
#include <string>
#include <vector>

#include "../../include/const_b200.h"

namespace cb {

struct TensorRef {
    std::string name;
    std::string idx;          // one character per mode, in reference order
};

struct Contraction {
    TensorRef out, lhs, rhs;
    std::string loops;        // outermost first
};

enum class Family { None, Ttmc3, Ttmc4, Mttkrp3, Network, Tree };

struct PlanDesc {
    TensorRef result;
    std::vector<TensorRef> inputs;                 // right-hand side of the expression
    std::vector<Contraction> tree;
    std::map<std::string, std::vector<int>> mode_orders;   // sparse inputs only
    std::map<char, int64_t> extents;
    const_dtype_t dtype = CONST_F32;

    // derived by check()
    std::vector<int> fused_loops;      // per contraction: number of fused loops removed from its result
    std::vector<int> reduced_order;    // per contraction: order of its result after fusion (0 for the last)

    // derived by match()
    Family family = Family::None;
    std::string sparse_name;           // chain: the CSF operand; network: U
    std::string sparse2_name;          // network: W
    std::vector<std::string> factor_names;   // chain: factor of level 1, 2, (3); network: V
    std::vector<int> ranks;            // chain: rank of each factor
    std::string error;                 // human-readable reason of the last failure
};

const_status_t parse_plan(const char *expression, const char *const *tree, int n_contractions,
                          const char *const *sparse_names, const int *const *mode_orders, int n_sparse,
                          const char *const *loop_orders, const const_extent_t *extents, int n_indices,
                          const_dtype_t dtype, PlanDesc &out);
const_status_t check_plan(PlanDesc &p);     // Sec. 3.2 constraints -> CONST_ERR_ILLEGAL_SCHEDULE
const_status_t match_plan(PlanDesc &p);     // kernel family      -> CONST_ERR_UNSUPPORTED
std::string schedule_cin(const PlanDesc &p); // loop_tree.cpp: concrete index notation of the schedule (Algorithm 1)

}  // namespace cb
