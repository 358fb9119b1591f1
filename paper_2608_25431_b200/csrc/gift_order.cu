// Multi-stream launch-order check (paper sec. 4.4, "Concurrency control") as a batch
// check over a recorded trace.
//
// The paper's monitor extends every ownership record with the last writer kernel and the
// last reader kernels of the segment, each a (stream, sequence number) pair, and keeps the
// last completed kernel per stream; a kernel is completed once a synchronisation operation
// on its stream follows its launch.  A reader may be launched only if the segment's last
// writer, when on another stream, has completed; a writer only if the last readers and the
// last writer on other streams have completed.
//
// Here the per-segment histories are given (launch order inside a segment is how the
// records accumulate), all segments are checked in parallel, one warp per segment with one
// lane per stream holding that stream's last reader, and every launch that breaks an
// invariant gets its flag bits set.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "gift_internal.cuh"

namespace {

constexpr int32_t NEVER = 0x7FFFFFFF;

// next_sync[e] = index of the first synchronisation of stream[e] after event e (NEVER if none).
// One CTA per stream runs a reverse minimum scan over the events in chunks of its size.
__global__ void next_sync_kernel(const uint8_t* __restrict__ kind, const int32_t* __restrict__ stream,
                                 uint32_t n_events, int32_t* __restrict__ next_sync)
{
    __shared__ int32_t warp_min[32];
    __shared__ int32_t carry_s;
    const int s = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
    if (tid == 0) carry_s = NEVER;
    __syncthreads();
    const uint32_t chunks = (n_events + blockDim.x - 1) / blockDim.x;
    for (uint32_t c = chunks; c-- > 0;) {
        // thread t of the chunk handles event base + (blockDim-1-t): reversed, so an inclusive
        // prefix minimum over t is a suffix minimum over events
        const uint32_t e = c * blockDim.x + (blockDim.x - 1 - tid);
        int32_t v = NEVER;
        bool mine = false;
        if (e < n_events && stream[e] == s) {
            mine = true;
            if (kind[e] == 1) v = (int32_t)e;
        }
        int32_t x = v;
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t y = __shfl_up_sync(0xFFFFFFFFu, x, o);
            if (lane >= o) x = min(x, y);
        }
        if (lane == 31) warp_min[wid] = x;
        __syncthreads();
        if (wid == 0) {
            int32_t w = lane < nw ? warp_min[lane] : NEVER;
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t y = __shfl_up_sync(0xFFFFFFFFu, w, o);
                if (lane >= o) w = min(w, y);
            }
            warp_min[lane] = w;
        }
        __syncthreads();
        const int32_t before = min(carry_s, wid ? warp_min[wid - 1] : NEVER);
        // exclusive of the event itself: a synchronisation at e does not complete a launch at e
        int32_t excl = __shfl_up_sync(0xFFFFFFFFu, x, 1);
        if (lane == 0) excl = NEVER;
        if (mine && kind[e] == 0) next_sync[e] = min(before, excl);
        __syncthreads();
        if (tid == 0) carry_s = min(carry_s, warp_min[nw - 1]);
        __syncthreads();
    }
}

__global__ void order_check_kernel(const int32_t* __restrict__ stream, uint32_t n_events, uint32_t n_streams,
                                   uint32_t n_segments, const int32_t* __restrict__ seg_ptr,
                                   const int32_t* __restrict__ seg_event, const uint8_t* __restrict__ seg_write,
                                   const int32_t* __restrict__ next_sync, uint32_t* __restrict__ flags)
{
    const int lane = threadIdx.x & 31;
    const uint32_t m = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (m >= n_segments) return;
    int32_t lw_stream = -1, lw_done = NEVER;      // last writer: its stream and when it completes
    bool has_lw = false;
    bool has_lr = false;                          // this lane's stream: last reader, and when it completes
    int32_t lr_done = NEVER;
    const int32_t a1 = seg_ptr[m + 1];
    int32_t a = seg_ptr[m];
    while (a < a1) {
        const int32_t e = seg_event[a];
        int32_t b = a + 1;
        while (b < a1 && seg_event[b] == e) b++;                     // all accesses of one launch
        if (e < 0 || (uint32_t)e >= n_events) { a = b; continue; }
        const int32_t s = stream[e];
        if (s < 0 || (uint32_t)s >= n_streams) { a = b; continue; }
        uint32_t f = 0;
        bool reads = false, writes = false;
        for (int32_t k = a; k < b; k++) {
            if (seg_write[k]) writes = true; else reads = true;
        }
        const bool lw_in_flight = has_lw && lw_stream != s && !(lw_done < e);
        if (lw_in_flight) f |= (reads ? 1u : 0u) | (writes ? 4u : 0u);
        if (writes) {
            const bool mine = has_lr && lane != s && !(lr_done < e);
            if (__any_sync(0xFFFFFFFFu, mine)) f |= 2u;
        }
        if (f != 0 && lane == 0) atomicOr(flags + e, f);
        const int32_t done = next_sync[e];
        if (writes) { has_lw = true; lw_stream = s; lw_done = done; }
        if (reads && lane == s) { has_lr = true; lr_done = done; }
        a = b;
    }
}

__global__ void order_summary_kernel(const uint32_t* __restrict__ flags, uint32_t n_events, uint32_t* summary)
{
    const uint32_t e = blockIdx.x * blockDim.x + threadIdx.x;
    const bool bad = e < n_events && flags[e] != 0;
    const uint32_t mask = __ballot_sync(0xFFFFFFFFu, bad);
    if (bad && (int)(threadIdx.x & 31) == __ffs(mask) - 1) {
        atomicAdd(summary, (uint32_t)__popc(mask));
        atomicMin(summary + 1, e);
    }
}

__global__ void order_init_kernel(uint32_t* summary)
{
    summary[0] = 0u;
    summary[1] = 0xFFFFFFFFu;
}

}  // namespace

extern "C" int gift_check_launch_order(gift_ctx* c, const gift_trace* t, uint32_t* flags, uint32_t* summary,
                                       void* stream)
{
    if (!c || !t || !summary) return GIFT_E_INVAL;
    if (t->n_streams == 0 || t->n_streams > 32) return GIFT_E_RANGE;
    if (t->n_events && (!t->kind || !t->stream || !flags)) return GIFT_E_INVAL;
    if (t->n_segments && (!t->seg_ptr || !t->seg_event || !t->seg_write)) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    if (t->n_events > c->order_cap) {
        CU_TRY(cudaDeviceSynchronize());
        cudaFree(c->d_next_sync);
        c->d_next_sync = nullptr;
        c->order_cap = 0;
        CU_TRY(cudaMalloc(&c->d_next_sync, (size_t)t->n_events * sizeof(int32_t)));
        c->order_cap = t->n_events;
    }
    order_init_kernel<<<1, 1, 0, st>>>(summary);
    c->launches++;
    if (t->n_events == 0) return GIFT_OK;
    CU_TRY(cudaMemsetAsync(flags, 0, (size_t)t->n_events * sizeof(uint32_t), st));
    next_sync_kernel<<<t->n_streams, 1024, 0, st>>>(t->kind, t->stream, t->n_events, c->d_next_sync);
    c->launches++;
    if (t->n_segments) {
        const uint64_t threads = (uint64_t)t->n_segments * 32;
        order_check_kernel<<<(uint32_t)((threads + 255) / 256), 256, 0, st>>>(
            t->stream, t->n_events, t->n_streams, t->n_segments, t->seg_ptr, t->seg_event, t->seg_write,
            c->d_next_sync, flags);
        c->launches++;
    }
    order_summary_kernel<<<(t->n_events + 255) / 256, 256, 0, st>>>(flags, t->n_events, summary);
    c->launches++;
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}
