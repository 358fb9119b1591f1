// Fused rule chain (paper sec. 4.3, rule steps 4 and 5, for the consecutive kernels of one
// forward pass): up to GIFT_CHAIN_MAX label rules applied one after another in ONE launch.
// Label maps are small (one int32 per token, block or page: a few hundred KiB), so a rule
// launched on its own costs its launch latency and nothing else; the chain pays that once.
//
// The launch is one thread-block cluster of 16 CTAs x 1024 threads (8 where the device cannot
// co-schedule 16).  Rule k+1 reads what rule
// k wrote, from any CTA, so the stages are separated by the cluster's hardware barrier
// (release on arrive, acquire on wait: the stage's global stores are visible to the whole
// cluster afterwards); inputs are read past L1 (ld.global.cg) so that no line cached before
// the barrier is used.  No grid-wide software barrier and no flag is spun on.
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gift_internal.cuh"
#include "gift_rules.cuh"

namespace cg = cooperative_groups;
using namespace gift;

namespace {

constexpr int CHAIN_CTAS_PORTABLE = 8;
constexpr int CHAIN_CTAS_LARGE = 16;      // needs the non-portable cluster size opt-in
constexpr int CHAIN_THREADS = 1024;
constexpr int MAX_DEVICES = 64;

struct ChainArgs {
    uint32_t n;
    uint32_t pad;
    RuleArgs r[GIFT_CHAIN_MAX];
};

__device__ __forceinline__ int32_t ld(const int32_t* p) { return __ldcg(p); }

// Every thread takes U outputs per pass and issues all their loads before it uses any: with
// 8 192 threads a map of 10^5 units is a handful of units per thread, and the stage then costs
// about one memory latency per dependent load instead of one per unit.  Conflicts are counted
// per thread and reported once per warp at the end of the stage.
constexpr int U = 8;

__device__ void stage_pointwise(const RuleArgs& r, uint32_t tid, uint32_t nthr)
{
    uint32_t n_conf = 0, first = 0xFFFFFFFFu;
    for (uint32_t base = tid; base < r.n_out; base += nthr * U) {
        JoinAcc acc[U];
#pragma unroll
        for (int u = 0; u < U; u++) acc[u].init();
        if (r.kind == GIFT_RULE_IDENTITY) {
            int32_t v[U];
#pragma unroll
            for (int u = 0; u < U; u++) {
                const uint32_t j = base + u * nthr;
                v[u] = j < r.n_out ? ld(r.in[0] + j) : GIFT_OWNER_PARAM;
            }
#pragma unroll
            for (int u = 0; u < U; u++) acc[u].add(v[u]);
        } else if (r.kind == GIFT_RULE_BROADCAST) {
            int32_t g[U], v[U];
#pragma unroll
            for (int u = 0; u < U; u++) {
                const uint32_t j = base + u * nthr;
                g[u] = j < r.n_out ? ld(r.gather + j) : -1;
            }
#pragma unroll
            for (int u = 0; u < U; u++) {
                const bool in_range = g[u] >= 0 && (uint32_t)g[u] < r.n_in0;
                v[u] = in_range ? ld(r.in[0] + g[u]) : GIFT_OWNER_CONFLICT;
            }
#pragma unroll
            for (int u = 0; u < U; u++) acc[u].add(v[u]);
        } else {   // ROWWISE
            for (uint32_t k = 0; k < r.n_in; k++) {
                if ((r.param_mask >> k) & 1u) {
                    const bool mislabelled = ld(r.in[k]) != GIFT_OWNER_PARAM;   // step 4: parameter operand
#pragma unroll
                    for (int u = 0; u < U; u++) acc[u].bad |= mislabelled;
                } else {
                    int32_t v[U];
#pragma unroll
                    for (int u = 0; u < U; u++) {
                        const uint32_t j = base + u * nthr;
                        v[u] = j < r.n_out ? ld(r.in[k] + j) : GIFT_OWNER_PARAM;
                    }
#pragma unroll
                    for (int u = 0; u < U; u++) acc[u].add(v[u]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; u++) {
            const uint32_t j = base + u * nthr;
            if (j < r.n_out) {
                const int32_t o = acc[u].result();
                r.out[j] = o;
                if (o == GIFT_OWNER_CONFLICT) { n_conf++; first = min(first, j); }
            }
        }
    }
    n_conf = __reduce_add_sync(0xFFFFFFFFu, n_conf);
    first = __reduce_min_sync(0xFFFFFFFFu, first);
    if ((tid & 31) == 0 && n_conf) {
        atomicAdd(r.viol, n_conf);
        atomicMin(r.viol + 1, first);
    }
}

// One warp per reduction segment, then the outputs that no segment covers.
__device__ void stage_segreduce(const RuleArgs& r, uint32_t tid, uint32_t nthr)
{
    const int lane = tid & 31;
    if (__ldcg(r.table_bad) != 0u) {
        // index arrays that are no valid CSR description: the launch as a whole is rejected
        for (uint32_t j = tid; j < r.n_out; j += nthr) r.out[j] = GIFT_OWNER_CONFLICT;
        if (tid == 0 && r.n_out) { r.viol[0] = r.n_out; r.viol[1] = 0u; }
        return;
    }
    for (uint32_t w = tid >> 5; w < r.n_seg; w += nthr >> 5) {
        const int32_t t0 = ld(r.seg_ptr + w), t1 = ld(r.seg_ptr + w + 1);
        const int32_t e0 = ld(r.src_ptr + w), e1 = ld(r.src_ptr + w + 1);
        JoinAcc acc;
        acc.init();
#pragma unroll 8
        for (int32_t t = t0 + lane; t < t1; t += 32) acc.add(ld(r.in[0] + t));
#pragma unroll 8
        for (int32_t e = e0 + lane; e < e1; e += 32) {
            const int32_t b = ld(r.src_idx + e);
            const bool in_range = b >= 0 && (uint32_t)b < r.n_in1;
            acc.add(in_range ? ld(r.in[1] + b) : GIFT_OWNER_CONFLICT);
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
    }
    const uint32_t head = (uint32_t)ld(r.seg_ptr);
    const uint32_t tail0 = (uint32_t)ld(r.seg_ptr + r.n_seg);
    const uint32_t n_extra = head + (r.n_out - tail0);
    for (uint32_t e = tid; e < n_extra; e += nthr) {
        const uint32_t j = e < head ? e : tail0 + (e - head);
        r.out[j] = GIFT_OWNER_CONFLICT;
        atomicAdd(r.viol, 1u);
        atomicMin(r.viol + 1, j);
    }
}

__global__ void __launch_bounds__(CHAIN_THREADS, 1)
rule_chain_kernel(const __grid_constant__ ChainArgs a)
{
    cg::cluster_group cl = cg::this_cluster();
    const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t nthr = gridDim.x * blockDim.x;
    if (tid < a.n) {
        a.r[tid].viol[0] = 0u;
        a.r[tid].viol[1] = 0xFFFFFFFFu;
    }
    // the index arrays of the reduction rules are inputs of the chain, so all of them are
    // checked up front (their flags are zero on entry and are put back to zero at the end)
    for (uint32_t k = 0; k < a.n; k++) {
        const RuleArgs& r = a.r[k];
        if (r.kind != GIFT_RULE_SEGREDUCE) continue;
        const bool bad = csr_tables_bad(r, tid, nthr);
        if (__any_sync(0xFFFFFFFFu, bad) && (tid & 31) == 0) atomicOr(r.table_bad, 1u);
    }
    cl.sync();
    for (uint32_t k = 0; k < a.n; k++) {
        const RuleArgs& r = a.r[k];
        if (r.kind == GIFT_RULE_SEGREDUCE) stage_segreduce(r, tid, nthr);
        else stage_pointwise(r, tid, nthr);
        cl.sync();
    }
    if (tid < a.n) *a.r[tid].table_bad = 0u;
}

}  // namespace

extern "C" int gift_propagate_chain(gift_ctx* c, const gift_rule* rules, const int32_t* const* const* in_maps,
                                    int32_t* const* outs, uint32_t n_rules, uint32_t* viol, void* stream)
{
    if (!c || !viol) return GIFT_E_INVAL;
    if (n_rules == 0) return GIFT_OK;
    if (!rules || !in_maps || !outs) return GIFT_E_INVAL;
    if (n_rules > GIFT_CHAIN_MAX) return GIFT_E_RANGE;
    ChainArgs a;
    memset(&a, 0, sizeof(a));
    a.n = n_rules;
    for (uint32_t k = 0; k < n_rules; k++) {
        const int rc = fill_rule_args(&rules[k], in_maps[k], outs[k], viol + 2 * k, a.r[k]);
        if (rc != GIFT_OK) return rc;
        a.r[k].table_bad = c->d_rule_flags + k;
        // The chain takes no snapshot: an input that is read at other indices than the one
        // written (the gather source, the block-owner map) must not overlap the stage's output.
        const gift_rule& g = rules[k];
        const int32_t* far = nullptr;
        uint32_t far_n = 0;
        if (g.kind == GIFT_RULE_BROADCAST) { far = in_maps[k][0]; far_n = g.n_in0; }
        if (g.kind == GIFT_RULE_SEGREDUCE) { far = in_maps[k][1]; far_n = g.n_in1; }
        if (far && far_n && g.n_out && ranges_overlap(far, (size_t)far_n * 4, outs[k], (size_t)g.n_out * 4))
            return GIFT_E_INVAL;
    }
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.blockDim = dim3(CHAIN_THREADS, 1, 1);
    cfg.stream = (cudaStream_t)stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    // Once per device: can a cluster of 16 CTAs of this kernel be co-scheduled?
    static int ctas_for_device[MAX_DEVICES];
    const int slot = c->device >= 0 && c->device < MAX_DEVICES ? c->device : -1;
    int ctas = slot >= 0 ? ctas_for_device[slot] : CHAIN_CTAS_PORTABLE;
    if (ctas == 0) {
        ctas = CHAIN_CTAS_PORTABLE;
        if (cudaFuncSetAttribute(rule_chain_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
            int n_clusters = 0;
            cfg.gridDim = dim3(CHAIN_CTAS_LARGE, 1, 1);
            attr.val.clusterDim.x = CHAIN_CTAS_LARGE;
            if (cudaOccupancyMaxActiveClusters(&n_clusters, rule_chain_kernel, &cfg) == cudaSuccess && n_clusters >= 1)
                ctas = CHAIN_CTAS_LARGE;
        }
        (void)cudaGetLastError();
        ctas_for_device[slot] = ctas;
    }
    cfg.gridDim = dim3(ctas, 1, 1);
    attr.val.clusterDim.x = ctas;
    CU_TRY(cudaLaunchKernelEx(&cfg, rule_chain_kernel, a));
    c->launches++;
    return GIFT_OK;
}
