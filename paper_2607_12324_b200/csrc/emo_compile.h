// Host-side compilation of an execution graph into the step programs the kernels interpret.
//
// The kernels give every group of 32 policies `lanes` cooperating warps.  Time is cut into steps;
// in one step every warp handles at most one node: it gathers the values of the node's
// predecessors (Eq. 1: C_v = t_v + max over predecessors of C_k), adds the node's duration and keeps
// the result in a register.  A value another warp (or a later, non-adjacent step of the same warp)
// needs is also written to a numbered exchange slot in shared memory.  All predecessors of a node
// are handled in strictly earlier steps and the warps of a group meet at a barrier after every
// step, so a slot is always written before it is read.  The backward pass (latest start times) runs
// the same machinery on the reversed graph.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

namespace emo {

constexpr uint32_t kNone = 0xFFFFFFFFu;
constexpr int kMaxSlotPreds = 6;      // slot operands one entry can name
constexpr int kMaxSlots = 250;        // exchange slots per policy group (8-bit ids)
constexpr int kMaxLanes = 32;

// entry word 2
constexpr uint32_t kValid = 1u, kRegPred = 2u, kWriteSlot = 4u, kTerminal = 8u, kAux = 0x80u;
constexpr int kNPredShift = 4;        // bits 4..6: number of slot operands
constexpr int kOutShift = 8;          // bits 8..15: slot written; bits 16..31: operand slots 4 and 5

struct Program {
    int lanes = 0, steps = 0, slots = 0, aux = 0, Lp = 0;
    std::vector<uint32_t> entries;    // [steps][lanes][4]: {policy row, node id, flags|out slot|operands 4-5, operand slots 0-3}
    std::vector<uint32_t> lat;        // [steps*lanes][Lp] durations of the scheduled node per level
    std::vector<double> energy;       // [steps*lanes][Lp], forward program only
};

struct HostGraph {
    int32_t n = 0, L = 0, rows = 0, depth = 0, max_span = 0;
    int64_t m = 0, T_worst = 0, T_best = 0;
    std::vector<int64_t> row_ptr;
    std::vector<int32_t> col;
    std::vector<int32_t> group;       // policy row of node v, -1 = none
};

// Builds the forward (backward = false) or backward program.  lanes <= 0 picks a value from the
// graph's shape.  Returns 0 or an EMO_E_* code and a message in err.
int compile_program(const HostGraph &g, const int64_t *lat, const double *energy, bool backward,
                    int lanes, int lookahead, Program &out, std::string &err);

int pick_lanes(int64_t n_ops, int depth);

}  // namespace emo
