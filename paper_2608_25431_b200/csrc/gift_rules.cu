// Label propagation, one rule per call (paper sec. 4.3, rule steps 4 and 5); the fused chain
// of several rules is in gift_chain.cu.
#include <cuda_runtime.h>
#include <stdint.h>

#include "gift_internal.cuh"
#include "gift_rules.cuh"

using namespace gift;

namespace {

__global__ void rule_pointwise_kernel(RuleArgs r)
{
    const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= r.n_out) return;
    JoinAcc acc;
    acc.init();
    if (r.kind == GIFT_RULE_IDENTITY) {
        acc.add(r.in[0][j]);
    } else if (r.kind == GIFT_RULE_BROADCAST) {
        const int32_t g = r.gather[j];
        if (g < 0 || (uint32_t)g >= r.n_in0) acc.bad = true; else acc.add(r.in[0][g]);
    } else {   // ROWWISE
        for (uint32_t k = 0; k < r.n_in; k++) {
            if ((r.param_mask >> k) & 1u) {
                if (r.in[k][0] != GIFT_OWNER_PARAM) acc.bad = true;   // step 4: parameter operand mislabelled
            } else {
                acc.add(r.in[k][j]);
            }
        }
    }
    const int32_t o = acc.result();
    r.out[j] = o;
    report_violation(r.viol, o == GIFT_OWNER_CONFLICT, j);
}

// One warp per reduction segment; outputs outside every segment become CONFLICT.  The rule's
// index arrays have been checked by rule_init_kernel: if they are no valid CSR description
// the launch as a whole is rejected (every output CONFLICT) and no index from them is used.
__global__ void rule_segreduce_kernel(RuleArgs r)
{
    const int lane = threadIdx.x & 31;
    const uint32_t gid = blockIdx.x * blockDim.x + threadIdx.x;
    if (*r.table_bad != 0u) {
        for (uint32_t j = gid; j < r.n_out; j += gridDim.x * blockDim.x) r.out[j] = GIFT_OWNER_CONFLICT;
        if (gid == 0 && r.n_out) { r.viol[0] = r.n_out; r.viol[1] = 0u; }
        return;
    }
    const uint32_t w = gid >> 5;
    if (w < r.n_seg) {
        const int32_t t0 = r.seg_ptr[w], t1 = r.seg_ptr[w + 1];
        const int32_t e0 = r.src_ptr[w], e1 = r.src_ptr[w + 1];
        JoinAcc acc;
        acc.init();
        for (int32_t t = t0 + lane; t < t1; t += 32) acc.add(r.in[0][t]);
        for (int32_t e = e0 + lane; e < e1; e += 32) {
            const int32_t b = r.src_idx[e];
            if (b < 0 || (uint32_t)b >= r.n_in1) acc.bad = true; else acc.add(r.in[1][b]);
        }
        acc.bad = __any_sync(0xFFFFFFFFu, acc.bad);
        acc.lo = __reduce_min_sync(0xFFFFFFFFu, acc.lo);
        acc.hi = __reduce_max_sync(0xFFFFFFFFu, acc.hi);
        const int32_t m = acc.result();
        __syncwarp();
        for (int32_t t = t0 + lane; t < t1; t += 32) r.out[t] = m;
        if (m == GIFT_OWNER_CONFLICT && lane == 0 && t1 > t0) {
            atomicAdd(r.viol, (uint32_t)(t1 - t0));
            atomicMin(r.viol + 1, (uint32_t)t0);
        }
    } else {
        // threads past the segments cover the outputs before the first and after the last segment
        const uint32_t extra = gid - r.n_seg * 32u;
        const uint32_t head = (uint32_t)r.seg_ptr[0];
        const uint32_t tail0 = (uint32_t)r.seg_ptr[r.n_seg];
        const uint32_t n_extra = head + (r.n_out - tail0);
        if (extra < n_extra) {
            const uint32_t j = extra < head ? extra : tail0 + (extra - head);
            r.out[j] = GIFT_OWNER_CONFLICT;
            atomicAdd(r.viol, 1u);
            atomicMin(r.viol + 1, j);
        }
    }
}

// Before the rule: the violation words start empty, and a SEGREDUCE rule's index arrays are
// checked (one block).
__global__ void rule_init_kernel(RuleArgs r)
{
    if (threadIdx.x == 0) {
        r.viol[0] = 0u;
        r.viol[1] = 0xFFFFFFFFu;
    }
    if (r.kind == GIFT_RULE_SEGREDUCE) {
        const bool bad = csr_tables_bad(r, threadIdx.x, blockDim.x);
        const int any = __syncthreads_or(bad ? 1 : 0);
        if (threadIdx.x == 0) *r.table_bad = any ? 1u : 0u;
    }
}

}  // namespace

extern "C" int gift_propagate_labels(gift_ctx* c, const gift_rule* rule, const int32_t* const* in_maps, int32_t* out,
                                     uint32_t* viol, void* stream)
{
    if (!c) return GIFT_E_INVAL;
    RuleArgs r;
    const int rc = fill_rule_args(rule, in_maps, out, viol, r);
    if (rc != GIFT_OK) return rc;
    r.table_bad = c->d_rule_flags + GIFT_CHAIN_MAX;      // the chain uses words 0 .. GIFT_CHAIN_MAX-1
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    // Rules read a snapshot: an input that the output overlaps and that is read at other
    // indices than the one written (the gather source, the block-owner map) is copied first.
    const int32_t* hazard = nullptr;
    uint32_t hazard_n = 0, hazard_slot = 0;
    if (rule->kind == GIFT_RULE_BROADCAST) { hazard = in_maps[0]; hazard_n = rule->n_in0; hazard_slot = 0; }
    if (rule->kind == GIFT_RULE_SEGREDUCE) { hazard = in_maps[1]; hazard_n = rule->n_in1; hazard_slot = 1; }
    if (hazard && hazard_n && rule->n_out &&
        ranges_overlap(hazard, (size_t)hazard_n * 4, out, (size_t)rule->n_out * 4)) {
        if (hazard_n > c->snapshot_cap) {
            CU_TRY(cudaDeviceSynchronize());
            cudaFree(c->d_snapshot);
            c->d_snapshot = nullptr; c->snapshot_cap = 0;
            CU_TRY(cudaMalloc(&c->d_snapshot, (size_t)hazard_n * 4));
            c->snapshot_cap = hazard_n;
        }
        CU_TRY(cudaMemcpyAsync(c->d_snapshot, hazard, (size_t)hazard_n * 4, cudaMemcpyDeviceToDevice, st));
        r.in[hazard_slot] = c->d_snapshot;
    }
    rule_init_kernel<<<1, rule->kind == GIFT_RULE_SEGREDUCE ? 1024 : 32, 0, st>>>(r);
    c->launches++;
    if (rule->kind == GIFT_RULE_SEGREDUCE) {
        const uint64_t threads = (uint64_t)rule->n_seg * 32u + rule->n_out;   // upper bound on uncovered outputs
        rule_segreduce_kernel<<<(uint32_t)((threads + 255) / 256) + 1, 256, 0, st>>>(r);
        c->launches++;
    } else if (rule->n_out) {
        rule_pointwise_kernel<<<(rule->n_out + 255) / 256, 256, 0, st>>>(r);
        c->launches++;
    }
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}
