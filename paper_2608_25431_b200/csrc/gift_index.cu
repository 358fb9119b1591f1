// Two-level ownership index (paper sec. 4.2) and the first three steps of a flow rule
// (paper sec. 4.3, rule generation).
//
// Level 1 maps a base address to a tensor record (base, shape, element size and the
// ownership-related dimensions "odim"); level 2 maps the subscripts of those dimensions to
// an owner.  Before a rule propagates labels it (1) finds the records of the kernel's
// arguments by base address, (2) checks the arguments against the recorded shapes and
// (3) checks that the tensors do not overlap unless they are meant to alias.  These are
// a handful of records per launch: plain host code.  What does run on the GPU is the
// expansion of level-2 records into one label per contiguous run of bytes, which is the
// form the segment calls consume (one ownership unit per page), so that an ownership
// slice such as C[1,2,:,0:8,:] of a 5-dimensional KV tensor becomes a paged segment whose
// page is the slice's run length.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "gift_internal.cuh"

namespace {

uint64_t rec_elems(const gift_tensor_rec* r)
{
    uint64_t n = 1;
    for (uint32_t d = 0; d < r->ndim; d++) n *= r->shape[d];
    return n;
}

bool rec_valid(const gift_tensor_rec* r)
{
    if (!r || r->ndim == 0 || r->ndim > GIFT_MAX_DIMS || r->elem_size == 0) return false;
    for (uint32_t d = 0; d < r->ndim; d++)
        if (r->shape[d] == 0) return false;
    return (r->odim_mask >> r->ndim) == 0;
}

struct ExpandArgs {
    uint32_t ndim, elem_size, odim_mask;
    uint64_t shape[GIFT_MAX_DIMS];
    uint64_t run_bytes, n_units;
    uint64_t sub_bytes;            // bytes that are guaranteed to lie in one ownership record
    uint32_t n_sub;                // pieces of sub_bytes per run
    const int32_t* owners;
    int32_t* out;
};

// One thread per run of run_bytes bytes.  The subscripts of an element, projected onto the
// ownership-related dimensions, give its level-2 record.  A run longer than one record's
// extent (eight slots of a block whose records are per slot) takes the label its records
// agree on, or CONFLICT if they differ.
__global__ void expand_owners_kernel(ExpandArgs a)
{
    const uint64_t u = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= a.n_units) return;
    int32_t label = 0;
    for (uint32_t k = 0; k < a.n_sub; k++) {
        uint64_t e = (u * a.run_bytes + (uint64_t)k * a.sub_bytes) / a.elem_size;
        uint64_t sub[GIFT_MAX_DIMS];
        for (int d = (int)a.ndim - 1; d >= 0; d--) {
            sub[d] = e % a.shape[d];
            e /= a.shape[d];
        }
        uint64_t idx = 0;
        for (uint32_t d = 0; d < a.ndim; d++)
            if ((a.odim_mask >> d) & 1u) idx = idx * a.shape[d] + sub[d];
        const int32_t l = a.owners[idx];
        if (k == 0) label = l;
        else if (l != label) label = GIFT_OWNER_CONFLICT;
    }
    a.out[u] = label;
}

// Secure swap space (paper sec. 4.5): blocks swapped to the monitor's own memory are not
// encrypted, but their ownership travels with them.
__global__ void swap_out_kernel(int32_t* owner_map, uint32_t n_units, const int32_t* __restrict__ units, uint32_t n,
                                int32_t* __restrict__ saved, uint32_t* viol)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int32_t u = units[i];
    if (u < 0 || (uint32_t)u >= n_units) {
        saved[i] = GIFT_OWNER_CONFLICT;
        atomicAdd(viol, 1u);
        atomicMin(viol + 1, i);
        return;
    }
    saved[i] = owner_map[u];
    owner_map[u] = GIFT_OWNER_NONE;          // the freed slot may not be read (sec. 4.2)
}

__global__ void swap_in_kernel(int32_t* owner_map, uint32_t n_units, const int32_t* __restrict__ units, uint32_t n,
                               const int32_t* __restrict__ saved, uint32_t* viol)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int32_t u = units[i];
    bool bad = u < 0 || (uint32_t)u >= n_units;
    if (!bad) {
        // a slot that still holds someone's data must not be overwritten by a swap-in
        const bool occupied = owner_map[u] != GIFT_OWNER_NONE;
        owner_map[u] = occupied ? GIFT_OWNER_CONFLICT : saved[i];
        bad = occupied;
    }
    if (bad) {
        atomicAdd(viol, 1u);
        atomicMin(viol + 1, i);
    }
}

__global__ void swap_viol_init_kernel(uint32_t* viol)
{
    viol[0] = 0u;
    viol[1] = 0xFFFFFFFFu;
}

}  // namespace

extern "C" {

int gift_labels_swap_out(gift_ctx* c, int32_t* owner_map, uint32_t n_units, const int32_t* units, uint32_t n,
                         int32_t* saved, uint32_t* viol, void* stream)
{
    if (!c || !viol || (n && (!owner_map || !units || !saved))) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    swap_viol_init_kernel<<<1, 1, 0, st>>>(viol);
    c->launches++;
    if (n) {
        swap_out_kernel<<<(n + 255) / 256, 256, 0, st>>>(owner_map, n_units, units, n, saved, viol);
        c->launches++;
    }
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}

int gift_labels_swap_in(gift_ctx* c, int32_t* owner_map, uint32_t n_units, const int32_t* units, uint32_t n,
                        const int32_t* saved, uint32_t* viol, void* stream)
{
    if (!c || !viol || (n && (!owner_map || !units || !saved))) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    swap_viol_init_kernel<<<1, 1, 0, st>>>(viol);
    c->launches++;
    if (n) {
        swap_in_kernel<<<(n + 255) / 256, 256, 0, st>>>(owner_map, n_units, units, n, saved, viol);
        c->launches++;
    }
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}

int gift_resolve_args(const gift_tensor_rec* recs, uint32_t n_rec, const gift_kernel_arg* args, uint32_t n_args,
                      int32_t* rec_of_arg, uint32_t* arg_status)
{
    if ((n_rec && !recs) || (n_args && (!args || !rec_of_arg || !arg_status))) return GIFT_E_INVAL;
    for (uint32_t i = 0; i < n_rec; i++)
        if (!rec_valid(&recs[i])) return GIFT_E_INVAL;
    for (uint32_t i = 0; i < n_args; i++) {
        rec_of_arg[i] = -1;
        arg_status[i] = GIFT_ARG_UNKNOWN;
        for (uint32_t k = 0; k < n_rec; k++) {                // step 1: record by base address
            if (recs[k].base != args[i].base) continue;
            rec_of_arg[i] = (int32_t)k;
            arg_status[i] = GIFT_ARG_OK;
            bool same = recs[k].ndim == args[i].ndim;         // step 2: expected shape
            for (uint32_t d = 0; same && d < recs[k].ndim; d++) same = recs[k].shape[d] == args[i].shape[d];
            if (!same) arg_status[i] |= GIFT_ARG_SHAPE;
            break;
        }
    }
    for (uint32_t i = 0; i < n_args; i++) {                   // step 3: unintended aliasing
        if (rec_of_arg[i] < 0) continue;
        const gift_tensor_rec* a = &recs[rec_of_arg[i]];
        const uint64_t a0 = a->base, a1 = a0 + rec_elems(a) * a->elem_size;
        for (uint32_t j = i + 1; j < n_args; j++) {
            if (rec_of_arg[j] < 0) continue;
            const gift_tensor_rec* b = &recs[rec_of_arg[j]];
            const uint64_t b0 = b->base, b1 = b0 + rec_elems(b) * b->elem_size;
            const bool overlap = a0 < b1 && b0 < a1;
            const bool intended = args[i].alias_group != 0 && args[i].alias_group == args[j].alias_group;
            if (overlap && !intended) {
                arg_status[i] |= GIFT_ARG_ALIAS;
                arg_status[j] |= GIFT_ARG_ALIAS;
            }
        }
    }
    return GIFT_OK;
}

int gift_slice_runs(const gift_tensor_rec* rec, const uint64_t* lo, const uint64_t* hi, uint64_t* run_bytes,
                    uint32_t* n_runs, int32_t* table, uint32_t table_cap)
{
    if (!rec_valid(rec) || !lo || !hi || !run_bytes || !n_runs) return GIFT_E_INVAL;
    const uint32_t nd = rec->ndim;
    for (uint32_t d = 0; d < nd; d++)
        if (lo[d] >= hi[d] || hi[d] > rec->shape[d]) return GIFT_E_RANGE;
    // the innermost dimensions taken whole, plus the range of the next one out, are contiguous
    int split = (int)nd - 1;
    uint64_t inner = rec->elem_size;                 // bytes of one step of dimension `split`
    while (split > 0 && lo[split] == 0 && hi[split] == rec->shape[split]) {
        inner *= rec->shape[split];
        split--;
    }
    const uint64_t run = inner * (hi[split] - lo[split]);
    if (run % 16 != 0) return GIFT_E_ALIGN;
    uint64_t count = 1;
    for (int d = 0; d < split; d++) count *= hi[d] - lo[d];
    if (count > 0x7FFFFFFFu) return GIFT_E_RANGE;
    *run_bytes = run;
    *n_runs = (uint32_t)count;
    if (!table) return GIFT_OK;
    if (table_cap < count) return GIFT_E_RANGE;
    uint64_t stride[GIFT_MAX_DIMS];
    uint64_t s = rec->elem_size;
    for (int d = (int)nd - 1; d >= 0; d--) {
        stride[d] = s;
        s *= rec->shape[d];
    }
    uint64_t sub[GIFT_MAX_DIMS];
    for (int d = 0; d < split; d++) sub[d] = lo[d];
    for (uint64_t r = 0; r < count; r++) {
        uint64_t off = lo[split] * stride[split];
        for (int d = 0; d < split; d++) off += sub[d] * stride[d];
        if (off % run != 0 || off / run > 0x7FFFFFFFu) return GIFT_E_ALIGN;    // a run must sit on a page boundary
        table[r] = (int32_t)(off / run);
        for (int d = split - 1; d >= 0; d--) {                                 // next outer subscript, row-major
            if (++sub[d] < hi[d]) break;
            sub[d] = lo[d];
        }
    }
    return GIFT_OK;
}

int gift_expand_owners(gift_ctx* c, const gift_tensor_rec* rec, uint64_t run_bytes, int32_t* unit_owner,
                       uint32_t n_units, void* stream)
{
    if (!c || !rec_valid(rec) || !rec->owners || !unit_owner || run_bytes == 0) return GIFT_E_INVAL;
    const uint64_t total = rec_elems(rec) * rec->elem_size;
    if (total % run_bytes != 0 || run_bytes % rec->elem_size != 0) return GIFT_E_ALIGN;
    if (total / run_bytes != n_units) return GIFT_E_RANGE;
    // below the innermost ownership-related dimension the bytes of one record are contiguous:
    // a run is either a part of one record or a whole number of records
    uint64_t below = rec->elem_size;
    int last_odim = -1;
    for (uint32_t d = 0; d < rec->ndim; d++)
        if ((rec->odim_mask >> d) & 1u) last_odim = (int)d;
    for (int d = (int)rec->ndim - 1; d > last_odim; d--) below *= rec->shape[d];
    uint64_t sub_bytes = run_bytes;
    uint32_t n_sub = 1;
    if (last_odim >= 0 && below % run_bytes != 0) {
        // the run spans several records: it must be a whole number of them
        if (run_bytes % below != 0 || run_bytes / below > 0xFFFFu) return GIFT_E_ALIGN;
        sub_bytes = below;
        n_sub = (uint32_t)(run_bytes / below);
    }
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    ExpandArgs a;
    memset(&a, 0, sizeof(a));
    a.ndim = rec->ndim; a.elem_size = rec->elem_size; a.odim_mask = rec->odim_mask;
    for (uint32_t d = 0; d < rec->ndim; d++) a.shape[d] = rec->shape[d];
    a.run_bytes = run_bytes; a.n_units = n_units; a.owners = rec->owners; a.out = unit_owner;
    a.sub_bytes = sub_bytes; a.n_sub = n_sub;
    expand_owners_kernel<<<(n_units + 255) / 256, 256, 0, (cudaStream_t)stream>>>(a);
    c->launches++;
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}

}  // extern "C"
