// Host-side compilation of an execution graph into the step programs the kernels interpret.
//
// The kernels give every group of 32 policies `lanes` cooperating warps.  Time is cut into steps;
// in one step every warp handles at most one node: it gathers the values of the node's
// predecessors (Eq. 1: C_v = t_v + max over predecessors of C_k), adds the node's duration and keeps
// the result in a register.  A value another warp (or a later, non-adjacent step of the same warp)
// needs is also written to a numbered exchange slot in shared memory.  All predecessors of a node
// are handled in strictly earlier steps.  The plain kernel runs the warps of a group in lockstep (a
// barrier after every step); the staged kernels let them drift: a reader polls the barrier of the
// slot it reads, the group meets only every `sync` steps, and a slot is reused only across such a
// meeting.  The backward pass (latest start times) runs the same machinery on the reversed graph.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

namespace emo {

constexpr uint32_t kNone = 0xFFFFFFFFu;
constexpr int kMaxSlotPreds = 6;      // slot operands one entry can name
constexpr int kMaxOperands = 6;       // operands per op; a node with more gets helper ops (3 was measured slower)
constexpr int kMaxSlots = 250;        // exchange slots per policy group (8-bit ids)
constexpr int kMaxLanes = 32;

// Program entry (32 bytes, 8 words): word 0 = row the entry addresses in the kernel's main per-node
// array (kNone for helper ops and idle entries); word 1 = flags; word 2 = operand slots 0..3,
// word 3 = operand slots 4..5 (8 bits each); word 4 = node id in the caller's numbering (kNone for
// helper ops and idle entries); word 5 = length of the run of plain entries that starts here (see
// emo_compile.cpp; 0 = not plain); word 6 = 1 when every slot operand was written before the last
// barrier of the group (no need to poll); word 7 unused.
constexpr int kEntryWords = 8;
constexpr uint32_t kValid = 1u, kRegPred = 2u, kWriteSlot = 4u, kTerminal = 8u, kAux = 0x80u;
constexpr int kNPredShift = 4;        // bits 4..6: number of slot operands
constexpr int kMaskShift = 8;         // bits 8..15: mask applied to the level byte (0 = node ignores the policy)
constexpr int kOutShift = 16;         // bits 16..23: slot written
constexpr int kOutParityShift = 24;   // bit 24: phase parity of the value written
constexpr int kOperandParityShift = 25;   // bits 25..30: phase parity of each operand's value
constexpr uint32_t kSimple = 0x80000000u;   // bit 31: simple entry (register operand only, no slot written, not terminal)
constexpr int kRunShift = 16;         // simple entries: bits 16..19 = length of the run of simple entries starting here
constexpr int kSyncSteps = 8;         // default distance (in steps) between two barriers of a group's warps

struct Program {
    int lanes = 0, steps = 0, slots = 0, aux = 0, Lp = 0;
    int sync = kSyncSteps;            // the warps of a group meet at a barrier every `sync` steps (a power of two)
    int64_t pruned = 0;               // edges dropped because they can never decide a maximum
    std::vector<uint32_t> entries;    // [steps][lanes][kEntryWords], see above
    std::vector<uint32_t> pos_of_node;   // [n] index (step*lanes + lane) of the entry that handles node v
    std::vector<uint32_t> rows;       // [steps][lanes] policy row whose level the entry reads (kNone: none)
    std::vector<uint32_t> groups;     // [steps][lanes] the node's group (its device, for time-interval policies) whether or not its
                                      // tables depend on the level; kNone: outside every policy
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
// row_in_other (optional, [n]): what to put into word 0 of a node's entry instead of its id.
// sync_steps (8, 16 or 32): distance between the barriers at which the warps of a group meet; a slot is
// reused only across such a barrier, so a larger distance costs slots and saves barriers.
int compile_program(const HostGraph &g, const int64_t *lat, const double *energy, bool backward,
                    int lanes, int lookahead, int sync_steps, const std::vector<uint32_t> *row_in_other,
                    Program &out, std::string &err);

int pick_lanes(int64_t n_ops, int depth);

// Target steps and list scheduling of ops, given by their operand lists in a topological order, onto
// `lanes` warps (<= 0: chosen from the shape).  step_of / warp_of give every op's place, prev_on_warp
// the op the same warp handled just before it (-1: none), steps the length of the schedule.
// gaps (optional, same shape as preds): the least distance in steps between an op and that operand
// (1 when absent).  With hard_gaps the distance is kept; without, it only shapes the target steps, so
// that the scheduler aims for it where the lanes have room.
int schedule_ops(const std::vector<std::vector<int32_t>> &preds, int lanes, int lookahead, std::vector<int32_t> &step_of,
                 std::vector<int32_t> &warp_of, std::vector<int32_t> &prev_on_warp, int32_t &steps, int &lanes_out,
                 std::string &err, const std::vector<std::vector<int32_t>> *gaps = nullptr, bool hard_gaps = true);

}  // namespace emo
