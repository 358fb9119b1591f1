// Validity of CSR pointer arrays that come from an untrusted launch description; compiles for
// host and device so that the host-side checks can run the same arithmetic without a GPU.
#pragma once
#include <stdint.h>

#include "gf128.cuh"

namespace gift {

// The index arrays of a SEGREDUCE rule come from the untrusted framework's launch
// description.  A pointer array is accepted only as a valid CSR description: first entry
// >= 0, non-decreasing, last entry <= limit.  csr_pair_ok checks one adjacent pair
// (lo = p[k], hi = p[k+1]) together with the two ends; a table is valid when every pair is.
GIFT_HD bool csr_pair_ok(int32_t lo, int32_t hi, bool first, bool last, uint32_t limit)
{
    if (hi < lo) return false;
    if (first && lo < 0) return false;
    if (last && (hi < 0 || (uint32_t)hi > limit)) return false;
    return true;
}

// The same for a table of one entry (no pair): 0 <= p[0] <= limit.
GIFT_HD bool csr_single_ok(int32_t p0, uint32_t limit)
{
    return p0 >= 0 && (uint32_t)p0 <= limit;
}

}  // namespace gift
