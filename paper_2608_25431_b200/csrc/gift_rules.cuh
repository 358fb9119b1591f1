// Label-rule pieces shared by the per-rule kernels and the fused rule chain (paper sec. 4.3,
// rule steps 4 and 5): the kernel argument block, the join over a set of labels and the
// violation report.  Not part of the public ABI.
#pragma once
#include <stdint.h>
#include <string.h>

#include "../../include/gift.h"
#include "gift_csr.cuh"

namespace gift {

struct RuleArgs {
    uint32_t kind, n_out, n_in, n_seg, n_in0, n_in1, n_src, param_mask;
    uint32_t* table_bad;            // SEGREDUCE: set to 1 before the rule runs if seg_ptr / src_ptr are malformed
    const int32_t* in[8];
    const int32_t* seg_ptr;
    const int32_t* src_ptr;
    const int32_t* src_idx;
    const int32_t* gather;
    int32_t* out;
    uint32_t* viol;
};

// The join over a set of labels is decided by three facts: was any label NONE or
// CONFLICT, the smallest user id seen and the largest one (PARAM is neutral).
struct JoinAcc {
    bool bad;
    int32_t lo, hi;
    __device__ __forceinline__ void init() { bad = false; lo = 0x7FFFFFFF; hi = -1; }
    __device__ __forceinline__ void add(int32_t l)
    {
        if (l <= GIFT_OWNER_NONE) bad = true;
        else if (l >= 0) { lo = min(lo, l); hi = max(hi, l); }
    }
    __device__ __forceinline__ int32_t result() const
    {
        if (bad) return GIFT_OWNER_CONFLICT;
        if (hi < 0) return GIFT_OWNER_PARAM;
        return lo == hi ? lo : GIFT_OWNER_CONFLICT;
    }
};

__device__ __forceinline__ void report_violation(uint32_t* viol, bool conflict, uint32_t j)
{
    const uint32_t m = __ballot_sync(__activemask(), conflict);
    if (conflict) {
        const int leader = __ffs(m) - 1;
        if ((int)(threadIdx.x & 31) == leader) {
            atomicAdd(viol, (uint32_t)__popc(m));
            atomicMin(viol + 1, j);      // the leader holds the smallest index of its warp
        }
    }
}

// Host: check a rule description and turn it into the kernel argument block.
inline int fill_rule_args(const gift_rule* rule, const int32_t* const* in_maps, int32_t* out, uint32_t* viol,
                          RuleArgs& r)
{
    if (!rule || !in_maps || !viol) return GIFT_E_INVAL;
    if (rule->n_out && !out) return GIFT_E_INVAL;
    memset(&r, 0, sizeof(r));
    r.kind = rule->kind; r.n_out = rule->n_out; r.n_in = rule->n_in; r.n_seg = rule->n_seg;
    r.n_in0 = rule->n_in0; r.n_in1 = rule->n_in1; r.n_src = rule->n_src; r.param_mask = rule->param_mask;
    r.seg_ptr = rule->seg_ptr; r.src_ptr = rule->src_ptr; r.src_idx = rule->src_idx; r.gather = rule->gather;
    r.out = out; r.viol = viol;
    uint32_t want_in = 1;
    switch (rule->kind) {
    case GIFT_RULE_IDENTITY: break;
    case GIFT_RULE_BROADCAST: if (!rule->gather && rule->n_out) return GIFT_E_INVAL; break;
    case GIFT_RULE_ROWWISE:
        if (rule->n_in < 1 || rule->n_in > 8) return GIFT_E_INVAL;
        want_in = rule->n_in;
        break;
    case GIFT_RULE_SEGREDUCE:
        if (rule->n_in != 2 || !rule->seg_ptr || !rule->src_ptr || (!rule->src_idx && rule->n_seg)) return GIFT_E_INVAL;
        want_in = 2;
        break;
    default: return GIFT_E_INVAL;
    }
    if (rule->n_in != want_in) return GIFT_E_INVAL;
    for (uint32_t k = 0; k < want_in; k++) {
        if (!in_maps[k]) return GIFT_E_INVAL;
        r.in[k] = in_maps[k];
    }
    return GIFT_OK;
}

#if defined(__CUDACC__)
// Every thread of the calling group checks its share of the pairs of both pointer arrays;
// returns true if this thread saw a malformed pair.
__device__ __forceinline__ bool csr_tables_bad(const RuleArgs& r, uint32_t tid, uint32_t nthr)
{
    bool bad = false;
    if (r.n_seg == 0) {
        if (tid == 0) bad = !csr_single_ok(r.seg_ptr[0], r.n_out) || !csr_single_ok(r.src_ptr[0], r.n_src);
        return bad;
    }
    for (uint32_t k = tid; k < r.n_seg; k += nthr) {
        bad |= !csr_pair_ok(r.seg_ptr[k], r.seg_ptr[k + 1], k == 0, k + 1 == r.n_seg, r.n_out);
        bad |= !csr_pair_ok(r.src_ptr[k], r.src_ptr[k + 1], k == 0, k + 1 == r.n_seg, r.n_src);
    }
    return bad;
}
#endif

inline bool ranges_overlap(const void* a, size_t na, const void* b, size_t nb)
{
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + nb && b0 < a0 + na;
}

}  // namespace gift
