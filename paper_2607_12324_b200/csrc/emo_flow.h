// Lane-stream programs: the compiled form of an execution graph that the 32-bit pass kernels walk.
//
// One schedule serves both passes.  Every node is placed on one of `lanes` warps (a lane) at one
// step; a lane's nodes, in step order, form its stream.  The forward pass (Eq. 1) walks every
// stream from its first entry to its last, the backward pass (latest starts) walks the same streams
// from the last entry to the first.  Streams are cut into stages of K steps (what the producer
// warps bring into shared memory at once) and stages into periods of `sync` steps (the warps of a
// policy group meet at a barrier where a period begins; exchange slots are reused only across such a
// barrier).
//
// Times are carried as unsigned 32-bit offsets from static lower bounds.  With dmin_v / dmax_v the
// smallest / largest entry of node v's duration row:
//   forward   lbES_v = max over predecessors of lbC_k (0 for a source), lbC_v = lbES_v + dmin_v,
//             eo_v = ES_v - lbES_v, co_v = C_v - lbC_v = eo_v + (t_v - dmin_v);
//             an operand k of v contributes co_k - (lbES_v - lbC_k), floored at 0
//   backward  Q_v = t_v + max over successors of Q_u (the longest tail from v's start), lbQin_v = max
//             over successors of lbQ_u, lbQ_v = lbQin_v + dmin_v, qin_v = (max over successors of Q_u)
//             - lbQin_v, qo_v = qin_v + (t_v - dmin_v)
//   slack_v = T - Q_v - ES_v = T - (lbQ_v + lbES_v) - (qin_v + co_v)
// The upper bounds (same recurrences with dmax) give the largest offset any policy can produce; the
// program exists only when every such spread fits 32 bits (Flow::ok32), and they prune operands
// that can never decide a maximum.
//
// The backward pass needs co_v of every node.  Along a stream it recovers it by subtraction: when
// entry i took its start from the lane's own previous value alone (co_{i-1} = eo_i), then
// co_{i-1} = co_i - (t_i - dmin_i).  Where that does not hold (several operands, or none) the
// forward pass pushes the lane's previous value to a restore list and the backward pass pops it.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

#include "emo_compile.h"

namespace emo {

constexpr int kFlowMaxLanes = 30;
constexpr int kFRecWords = 8;      // forward record: flags, out slot, out tag / correction, pool offset, first operand
                                   // (3 words), correction of the lane's previous value
constexpr int kBRecWords = 16;     // backward record: flags, out slot, out tag / correction, pool offset, A_v (2 words),
                                   // node id, correction of the lane's previous value, first operand (3 words), spare,
                                   // second operand (3 words), spare; further operands sit in the pool
constexpr int kOpWords = 3;        // operand descriptor: slot offset | kind bits, tag, delta
constexpr int kHdrWords = 8;       // per (stage, lane): word 0 = forward segments (bits 0..7) | backward segments (8..15)
                                   // | entries (16..23); word 4 pushes, word 5 first restore row inside the stage,
                                   // word 6 first restore row of the stage; the rest spare
constexpr int kFlowMaxStage = 32;  // most steps of a stage
constexpr int kFlowRun = 8;        // most simple entries of one segment (their look-ups are issued together)
constexpr int kSegBytes = 40;      // segment bytes per (stage, lane) and direction: at most K + K / sync
// segment byte: bits 0..3 simple entries in the run, then
constexpr uint32_t kSegRunMask = 15u;
constexpr uint32_t kSegSpecial = 16u;   // an entry that needs its record comes first
constexpr uint32_t kSegBarrier = 32u;   // the group meets before this segment (a period begins)
constexpr uint32_t kSegIn = 64u;        // backward run: every entry folds in one settled single-reader slot
constexpr uint32_t kSegOut = 128u;      // backward run: every entry writes one settled single-reader slot

// forward record word 0 (a plain entry has kF_HasReg alone)
constexpr uint32_t kF_HasReg = 1u << 8;     // starts from the lane's previous value
constexpr uint32_t kF_RegDelta = 1u << 9;   // ... after a correction (record word 7)
constexpr uint32_t kF_OutTag = 1u << 10;    // writes a tagged slot (value + tag, polled by readers)
constexpr uint32_t kF_OutSet = 1u << 11;    // writes a settled slot (value only, read after a barrier)
constexpr uint32_t kF_Terminal = 1u << 12;  // node without successors: candidate for the makespan
constexpr uint32_t kF_Push = 1u << 13;      // the lane's previous value goes to the restore list
constexpr uint32_t kF_OutAcc = 1u << 14;    // the settled slot is shared: the value is folded in with a maximum
constexpr int kF_NopsShift = 16;            // bits 16..31: slot operands
// backward record word 0
constexpr uint32_t kB_HasReg = 1u, kB_RegDelta = 2u, kB_OutTag = 4u, kB_OutSet = 8u, kB_Pop = 16u, kB_OutAcc = 32u;
// A simple backward entry continues from the lane's previous value (corrected by word 7), reads at
// most one slot and writes at most one, both settled with a single reader (so the value is stored
// already corrected and the reader resets the slot); word 3 then holds the operand's slot offset.
constexpr uint32_t kB_Simple = 64u;
constexpr int kB_NopsShift = 16;
// operand descriptor word 0
constexpr uint32_t kOpNoPoll = 1u << 31;    // written before the group's last barrier: no polling
constexpr uint32_t kOpWord = 1u << 30;      // a settled slot (4 bytes per policy) instead of a tagged one (8)
constexpr uint32_t kOpClear = 1u << 29;     // a settled slot with a single reader: the reader resets it to 0
constexpr uint32_t kOpOffMask = (1u << 29) - 1u;


// ---- spine programs -------------------------------------------------------------------------------
// A second form of the same schedule for the kernels of emo_spine.cuh.  A lane's consecutive entries
// whose only live link in both directions is the lane itself form a segment: along it completion
// offsets are running sums, and co_v + qin_v (hence T - Q_v - ES_v relative to A_v) is one number for
// all members.  Per stage the program lists the segments (for the warps that do the look-ups, sums,
// stores) and, per direction, one operation per segment for the single warp that carries the
// recurrence of a policy group (the spine): the maximum of two value slots (corrected), plus the
// segment's sum, written to the lane's slot and to a published slot.  A node with more operands gets
// merge operations in front.  Backward, a value that a node of a much earlier stage reads (two stages
// or more: a launch node and its kernels) is folded by the storing warps into a slot of that reader.
constexpr int kSpOpWordsF = 8;        // a0, d0, a1, d1, lane slot, published slot, sum offset, flags | push row << 8 | push row in the
                                      // paired numbering << 20 (both relative to the stage's base); terminal bounds are taken in order
constexpr int kSpOpWordsB = 12;       // the same eight (flags | pop row << 8), then: slot to clear, lane's completion slot, where the head's
                                      // tail goes (beside X if members are folded, else nowhere), where it goes when all tails are kept
constexpr int kSpSegWords = 4;        // lane | first position << 8 | members << 16 | flags << 24, sum offset, A_v low, high
constexpr int kSpMemWords = 8;        // node (kNone: unused position), fold slot, fold correction, position word, A_v low, high, lbES_v low, high
// position word (one per lane position of a stage): bit 0 = first member of its segment, bit 1 = last member,
// bits 4..15 = index of the segment in the stage's list, bits 16..31 = offset of the segment's sum in 128-byte units
constexpr uint32_t kSpPos_First = 1u, kSpPos_Last = 2u;
constexpr uint32_t kSp_NoSum = 1u;    // operation flags: the segment's sum is zero / a merge operation
constexpr uint32_t kSp_Push = 2u;     // forward: the lane's previous value goes to the restore list; backward: it is popped
constexpr uint32_t kSp_Terminal = 4u; // forward: the segment's last node has no successor
constexpr uint32_t kSpSeg_PreF = 1u, kSpSeg_PreB = 2u, kSpSeg_Fold = 4u;   // segment flags

struct SpineDir {
    int slots = 0;                    // value slots of a policy group (128 bytes each)
    int max_ops = 0;
    std::vector<uint32_t> n_ops;      // [stages]
    std::vector<uint32_t> ops;        // [stages][max_ops][kSpOpWordsF | kSpOpWordsB]
};

struct Spine {
    bool ok = false;
    int max_segs = 0, max_pool = 0;
    int acc_words = 0;                // 4-byte words per policy that the sums / results of one stage take
    int acc_words_all = 0;            // the same when every segment's head tail is kept (one more word per segment, behind the others)
    int64_t pushes = 0;
    int64_t segments = 0;
    std::vector<uint32_t> n_segs;     // [stages]
    std::vector<uint32_t> seg;        // [stages][max_segs][kSpSegWords]
    std::vector<uint32_t> mem;        // [stages][lanes * K][kSpMemWords]
    std::vector<uint32_t> posw;       // [stages][lanes * K] position words
    std::vector<uint64_t> pool;       // [stages][max_pool] lbC of terminal nodes
    std::vector<int64_t> push_base;   // [stages + 1]
    // the same restore rows numbered as a lane-stream program with stages of pair_K steps numbers them (per stage the
    // lanes in order, a lane's rows by position): the forward spine kernel can then feed the lane-stream backward kernel
    int pair_K = 0;
    bool pair_ok = false;
    std::vector<int64_t> pair_base;   // [stages] smallest such row of the stage's pushes
    SpineDir f, b;
};

struct FlowDir {
    int slots_tag = 0, slots_set = 0;   // tagged slots (256 bytes per group) and settled slots (128 bytes)
    int pool_stride = 4;                // words of operand pool per stage
    int64_t pruned = 0;                 // edges that can never decide a maximum in this direction
    std::vector<uint32_t> rec;          // [stages][lanes][K][kFRecWords | kBRecWords]
    std::vector<uint32_t> pool;         // [stages][pool_stride]
    std::vector<uint8_t> seg;           // [stages][lanes][kSegBytes] segment bytes in walking order
};

struct Flow {
    bool ok32 = false;                  // every spread fits 32 bits: the program below exists
    int lanes = 0, K = 0, sync = 0, stages = 0, steps = 0, Lp = 0;
    int64_t entries = 0;                // scheduled nodes
    int64_t pushes = 0;                 // restore rows per policy, all stages (the lanes' final values follow)
    std::vector<uint32_t> hdr;          // [stages][lanes][kHdrWords]
    std::vector<uint32_t> rows;         // [stages][lanes][K] policy row read by the entry, kNone = none
    std::vector<uint32_t> node;         // [stages][lanes][K] node id, kNone = unused position
    std::vector<uint32_t> step;         // [stages][lanes][K] step of the entry (host-side inspection)
    std::vector<uint32_t> tabF;         // [stages][lanes][K][Lp][3]: t - dmin, energy high word, low word
    std::vector<uint32_t> tabB;         // [stages][lanes][K][Lp]: t - dmin
    std::vector<int64_t> lbes;          // [stages][lanes][K] lbES_v (for the ES and LS outputs)
    std::vector<uint32_t> dmin;         // [stages][lanes][K] smallest entry of the node's duration row (time-interval policies)
    std::vector<uint32_t> grp;          // [stages][lanes][K] the node's group whether or not its tables depend on the level (kNone: none)
    std::vector<int64_t> push_base;     // [stages + 1] first restore row of every stage
    FlowDir f, b;
    Spine spine;                      // filled when the compiler is asked for it
};


// What the spine back-end takes from the compiler's analysis (all indexed as in compile_flow).
struct SpineIn {
    int32_t n = 0;
    int lanes = 0, K = 0, stages = 0, L = 0;
    const std::vector<int64_t> *pp = nullptr, *sp = nullptr;          // predecessor / successor CSR (deduplicated)
    const std::vector<int32_t> *pc = nullptr, *sc = nullptr;
    const std::vector<char> *liveF = nullptr, *liveB = nullptr;       // per predecessor-CSR edge
    const std::vector<char> *constant = nullptr;                      // node's tables do not depend on the level
    const std::vector<int64_t> *lbES = nullptr, *lbC = nullptr, *lbQin = nullptr, *lbQ = nullptr;
    const std::vector<int32_t> *step_of = nullptr, *lane_of = nullptr, *prev_on_lane = nullptr, *next_on_lane = nullptr, *pos_of = nullptr;
    const double *energy = nullptr;                                   // [n][L]
    int pair_K = 0;                                                   // stage length of the lane-stream program to pair with (0: none)
};
int build_spine(const SpineIn &in, Spine &out, std::string &err);

// Compiles g into a lane-stream program.  Returns EMO_OK with out.ok32 = false when the 32-bit
// representation does not apply (spread too large, too many lanes); other codes are errors.
int compile_flow(const HostGraph &g, const int64_t *lat, const double *energy, int lanes, int lookahead,
                 int K, int sync, Flow &out, std::string &err, bool spine = false, int pair_K = 0);

}  // namespace emo
