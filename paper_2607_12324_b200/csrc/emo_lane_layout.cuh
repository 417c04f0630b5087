// Program layout and small PTX helpers of the staged pass kernel emo_pass_lane (sm_100a).
//
// The program comes in a layout of its own (built at load time from the step program):
//   entry  [Q][8 words]  word 0 = row of the per-node store (forward: row of the earliest-start
//                        spill; backward: node id) or kNone; word 1 = out slot (bits 0..7, 255 =
//                        none) | number of slot operands (bits 8..10) | terminal (bit 11) | phase
//                        parity of the value written (bit 12) and of each operand (bits 13..18) |
//                        idle (bit 19) | length of the run of plain entries that starts here
//                        (bits 20..23; see emo_compile.cpp) | every slot operand was written before
//                        the group's last barrier, none needs polling (bit 24); word 2 = mask applied to the lane's running value (0 =
//                        start from 0, ~0 = continue from the lane's last node); word 3 = operand
//                        slots 0..3; word 4 = operand slots 4..5; word 5 = node id
//   table  [Q][Lp]       forward: {duration, high word of the energy, low word} in 12 bytes per
//                        level; backward: duration in 4 bytes.  Rows of nodes that ignore the policy
//                        hold one value Lp times.
// Q = padded steps x lanes; the padding steps are idle entries, so every stage holds whole steps.
// Included only by emo_lib.cu.
#pragma once
#include "emo_pass_staged.cuh"

constexpr int kLaneStepPad = 32;                 // programs are padded to a multiple of this many steps (the longest stage)
constexpr unsigned kLaneNoSlot = 255u;
constexpr unsigned kLaneNpShift = 8, kLaneTerminal = 0x800u, kLaneOutParShift = 12, kLaneOpParShift = 13, kLaneIdle = 1u << 19, kLaneRunShift = 20, kLaneSettled = 1u << 24;

// offsets of the areas of one stage (records first, then what emo_produce addresses)
struct LaneStage {
    unsigned off_tab;                           // entries start at 0
};

struct LaneParams {
    StagedParams sp;
    LaneStage st;
    unsigned tab_entry;                         // bytes of one entry's table row
};

__device__ __forceinline__ long long emo_lds_s64(unsigned a)
{
    long long v;
    asm volatile("ld.shared.s64 %0, [%1];" : "=l"(v) : "r"(a));
    return v;
}
// the value when cond holds, else 0 (no access)
__device__ __forceinline__ long long emo_lds_s64_if(unsigned a, bool cond)
{
    long long v = 0;
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p ld.shared.s64 %0, [%1];\n\t}" : "+l"(v) : "r"(a), "r"((unsigned)cond));
    return v;
}
__device__ __forceinline__ void emo_sts_s64(unsigned a, long long v)
{
    asm volatile("st.shared.s64 [%0], %1;" ::"r"(a), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned emo_lds_u8(unsigned a)
{
    unsigned v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}

// st.global / st.shared under a predicate (no branch): the store happens when row != kNone and ok != 0
__device__ __forceinline__ void emo_stg_row_if(long long *base, unsigned row, unsigned pitch_bytes, long long v, unsigned ok)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .u64 a;\n\t"
        "setp.ne.u32 q, %4, 0;\n\t"
        "setp.ne.and.u32 p, %1, 0xFFFFFFFF, q;\n\t"
        "mad.wide.u32 a, %1, %2, %0;\n\t"
        "@p st.global.s64 [a], %3;\n\t}"
        ::"l"(base), "r"(row), "r"(pitch_bytes), "l"(v), "r"(ok)
        : "memory");
}
__device__ __forceinline__ void emo_sts_s64_if(unsigned a, long long v, unsigned id, unsigned none)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, %3;\n\t@p st.shared.s64 [%0], %1;\n\t}" ::"r"(a), "l"(v), "r"(id), "r"(none)
                 : "memory");
}


