// Work plan of evo_validate: which tensors share a reference ("sets"), and which contiguous
// run of (set, tile) items each persistent CTA walks.  Built on the host per call, read by
// the kernels.  The records below are the device-side layout.
#pragma once

#include <stdint.h>

#include <string>
#include <vector>

#include "evo.h"

namespace evo {

constexpr int kThreads = 256;                   // consumer threads per CTA of the first pass (8 warps)
constexpr int kWarps = kThreads / 32;
constexpr int kBlock = kThreads + 32;           // plus one producer warp that issues the bulk copies
constexpr int kMaxK = 32;                       // members of one set (more are split into several sets)
constexpr int kEpt = 16;                        // elements per consumer thread per tile
constexpr int kTileElems = kEpt * kThreads;     // 4096 elements of every tensor per tile (16 KiB fp32, 8 KiB fp16/bf16)

struct Acc {                 // partial result of one tensor (40 bytes)
    unsigned long long mism;
    unsigned long long nonfin;
    double sse;
    uint32_t max_abs;        // binary32 bit patterns of non-negative values: unsigned order == float order
    uint32_t max_rel;
    uint32_t flags;
    uint32_t pad;
};

struct SetRec {              // tensors sharing one reference
    const void* ref;
    uint64_t n;
    uint32_t member_off;     // first entry in members[]
    uint32_t k;
    uint32_t dtype;
    uint32_t vec_ok;         // reference and all members 16-byte aligned
    uint32_t cta_first;      // CTAs that hold partial records of this set: [cta_first, cta_last]
    uint32_t cta_last;       // (first > last: none)
};

struct MemberRec {
    const void* cand;
    uint32_t desc;           // index of the caller's descriptor / result
    uint32_t set;
};

struct CtaRange {            // items [(s_begin, t_begin), (s_end, t_end)) with t_end exclusive inside s_end
    uint64_t t_begin;
    uint64_t t_end;
    uint32_t s_begin;
    uint32_t s_end;          // inclusive; s_begin > s_end: empty range
    uint32_t part_base;      // first partial record of this CTA
    uint32_t first_member;   // member_off of s_begin
};

// Bytes per element of every type a plan can hold (0: not a type).
inline uint32_t dtype_bytes(int dt) {
    switch (dt) {
        case EVO_F32: case EVO_I32: case EVO_U32: return 4;
        case EVO_F16: case EVO_BF16: return 2;
        case EVO_I64: case EVO_F64: return 8;
        case EVO_U8: return 1;
        default: return 0;
    }
}
constexpr uint32_t kFloatTypes = (1u << EVO_F32) | (1u << EVO_F16) | (1u << EVO_BF16);
constexpr uint32_t kIntTypes = (1u << EVO_I32) | (1u << EVO_I64) | (1u << EVO_U8);
constexpr uint32_t kWordTypes = (1u << EVO_I32) | (1u << EVO_U32);      // what a regenerated stream can be compared as

struct Plan {
    std::vector<SetRec> sets;
    std::vector<MemberRec> members;      // ordered by set
    std::vector<CtaRange> ranges;        // one per CTA of pass 1
    std::vector<uint32_t> group_off;     // n_group + 1 offsets into group_desc (empty without verdicts)
    std::vector<uint32_t> group_desc;    // descriptor indices ordered by candidate id
    uint32_t n_parts = 0;                // partial records pass 1 writes
    uint64_t total_tiles = 0;
};

// Checks the arguments of evo_validate and builds the plan for at most `max_ctas` CTAs.
// Pure host code (no CUDA call).  Returns EVO_OK or an EVO_ERR_* with `err` set.
int build_plan(const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs, uint64_t n_desc,
               int dtype, float atol, float rtol, bool want_groups, uint64_t n_group, uint32_t max_ctas,
               Plan* plan, std::string* err, uint32_t accepted_types = kFloatTypes);

}  // namespace evo
