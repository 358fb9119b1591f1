// libgift: context, keys and the segment entry points (see include/gift.h).  The kernels of
// the segment calls are in gift_seg.cuh.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "../../include/gift.h"
#include "gift_core.cuh"

using namespace gift;

#define GIFT_VERSION 200u   // 0.2.0

#include "gift_internal.cuh"
#include "gift_seg.cuh"

static thread_local char g_error_detail[384] = "";

// Keeps the newest failure first and the one before it behind, so that an error met in a
// clean-up path is still visible when a later call trips over it.
void gift_note_cuda_error(cudaError_t e, const char* file, int line)
{
    const char* base = file;
    for (const char* p = file; *p; p++)
        if (*p == '/') base = p + 1;
    char prev[160];
    snprintf(prev, sizeof(prev), "%s", g_error_detail);
    char* cut = strstr(prev, "; before that: ");
    if (cut) *cut = 0;
    snprintf(g_error_detail, sizeof(g_error_detail), "%s (%s) at %s:%d%s%s", cudaGetErrorName(e), cudaGetErrorString(e),
             base, line, prev[0] ? "; before that: " : "", prev);
}

namespace {

// ---------------------------------------------------------------------------
// tables and keys
// ---------------------------------------------------------------------------

__global__ void init_t0_kernel(uint32_t* t0, uint8_t* isbox)
{
    t0[threadIdx.x] = t0_entry(threadIdx.x);
    isbox[sbox_entry(threadIdx.x)] = (uint8_t)threadIdx.x;      // the S-box is a permutation
}

// Four threads per user: each derives the key schedule and H, thread m builds
// level m of the power table, thread 0 also stores the hot record.
__global__ void key_setup_kernel(const uint32_t* __restrict__ t0, const int32_t* __restrict__ ids,
                                 const uint8_t* __restrict__ keys, uint32_t n, KeyHot* hot, u128* pow)
{
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t i = g / POW_LEVELS;
    const int m = (int)(g % POW_LEVELS);
    if (i >= n) return;
    PlainTab tb;
    tb.t0 = t0;
    uint32_t key[4];
    const Block kb = load_block(keys + 16 * (size_t)i);
    key[0] = kb.d[0]; key[1] = kb.d[1]; key[2] = kb.d[2]; key[3] = kb.d[3];
    KeyHot rec;
    u128 h;
    derive_key_hot(tb, key, &rec, &h);
    const uint32_t u = (uint32_t)ids[i];
    build_pow_level(h, m, pow + (size_t)u * (POW_LEVELS * 256) + m * 256);
    if (m == 0) hot[u] = rec;
}

__global__ void key_clear_kernel(const int32_t* __restrict__ ids, uint32_t n, KeyHot* hot, u128* pow)
{
    const uint32_t i = blockIdx.x;
    if (i >= n) return;
    const uint32_t u = (uint32_t)ids[i];
    uint32_t* h = reinterpret_cast<uint32_t*>(hot + u);
    for (uint32_t k = threadIdx.x; k < sizeof(KeyHot) / 4; k += blockDim.x) h[k] = 0u;
    uint32_t* p = reinterpret_cast<uint32_t*>(pow + (size_t)u * (POW_LEVELS * 256));
    for (uint32_t k = threadIdx.x; k < POW_LEVELS * 256 * 4; k += blockDim.x) p[k] = 0u;
}

// ---------------------------------------------------------------------------
// host side of the segment calls
// ---------------------------------------------------------------------------

template <int MODE, int NT, bool FUSED, bool PEEL>
int launch_crypt_t(gift_ctx* c, const CallArgs& a, cudaStream_t st)
{
    constexpr size_t smem = crypt_smem_bytes<NT, FUSED>();
    constexpr int MAX_DEV = 64;
    static bool configured[MAX_DEV];
    auto kern = crypt_kernel<MODE, NT, FUSED, PEEL>;
    if (c->device < 0 || c->device >= MAX_DEV || !configured[c->device]) {
        CU_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        if (c->device >= 0 && c->device < MAX_DEV) configured[c->device] = true;
    }
    const bool timed = c->timing && c->ev && c->n_timed < MAX_TIMED;
    if (timed) CU_TRY(cudaEventRecord(c->ev[2 * c->n_timed], st));
    kern<<<c->num_sms, CRYPT_THREADS, smem, st>>>(a, c->d_t0);
    if (timed) {
        CU_TRY(cudaEventRecord(c->ev[2 * c->n_timed + 1], st));
        c->n_timed++;
    }
    c->launches++;
    return GIFT_OK;
}

// fused: the single-launch form (always with the first row peeled: its pieces are short).
// short_segments: the table's segments are small on average, so pieces are short too.
template <int MODE>
int launch_crypt(gift_ctx* c, const CallArgs& a, cudaStream_t st, bool fused, bool short_segments)
{
    if (fused)
        return c->tables == 4 ? launch_crypt_t<MODE, 4, true, true>(c, a, st) : launch_crypt_t<MODE, 2, true, true>(c, a, st);
    if (short_segments)
        return c->tables == 4 ? launch_crypt_t<MODE, 4, false, true>(c, a, st) : launch_crypt_t<MODE, 2, false, true>(c, a, st);
    return c->tables == 4 ? launch_crypt_t<MODE, 4, false, false>(c, a, st) : launch_crypt_t<MODE, 2, false, false>(c, a, st);
}

// The optional overlap check (GIFT_CTX_CHECK_OVERLAP): fills sc->overlap before the plan.
int launch_overlap_check(gift_ctx* c, SegScratch* sc, const CallArgs& a, cudaStream_t st)
{
    if (a.page_table == nullptr) {
        if (a.nseg > 65536u) return GIFT_E_RANGE;                // all pairs: bounded
        overlap_flat_kernel<<<(a.nseg + OVL_TILE - 1) / OVL_TILE, OVL_TILE, 0, st>>>(a, sc->overlap);
        c->launches++;
        return GIFT_OK;
    }
    const uint64_t n_phys = a.buf_bytes / a.page_bytes;           // physical pages that lie inside the buffer
    if (n_phys > ((uint64_t)1 << 28)) return GIFT_E_RANGE;
    if (n_phys > c->claim_cap) {
        CU_TRY(cudaDeviceSynchronize());
        CU_NOTE(cudaFree(c->d_claim));
        c->d_claim = nullptr; c->claim_cap = 0;
        CU_TRY(cudaMalloc(&c->d_claim, (size_t)n_phys * sizeof(int32_t)));
        c->claim_cap = n_phys;
    }
    if (n_phys) CU_TRY(cudaMemsetAsync(c->d_claim, 0xFF, (size_t)n_phys * sizeof(int32_t), st));
    CU_TRY(cudaMemsetAsync(sc->overlap, 0, a.nseg, st));
    overlap_paged_kernel<<<(a.nseg + 7) / 8, 256, 0, st>>>(a, c->d_claim, sc->overlap);
    c->launches++;
    return GIFT_OK;
}

constexpr uint64_t SHORT_SEGMENT_BYTES = 4096;

template <int MODE>
int seg_call(gift_ctx* c, SegScratch* sc, const void* src, void* dst, uint64_t buf_bytes, const gift_seg* segs,
             uint32_t nseg, uint32_t seg_base, const gift_pages* pages, const gift_labels* labels, uint8_t* tags,
             uint32_t* status, cudaStream_t st, bool allow_fused)
{
    CallArgs a;
    memset(&a, 0, sizeof(a));
    a.src = (const uint8_t*)src;
    a.dst = (uint8_t*)dst;
    a.buf_bytes = buf_bytes;
    a.segs = segs;
    a.nseg = nseg;
    if (pages) { a.page_table = pages->table; a.n_pages = pages->n; a.page_bytes = pages->page_bytes; }
    if (labels) { a.owner_map = labels->owner_map; a.n_units = labels->n_units; a.unit_bytes = labels->unit_bytes; }
    a.tags = tags;
    a.aad = c->aad ? c->aad + 16 * (size_t)seg_base : nullptr;
    a.status = status;
    a.hot = c->d_hot;
    a.pow = c->d_pow;
    a.max_users = c->max_users;
    a.wprefix = sc->wprefix;
    a.acc = sc->acc;
    a.ticket = sc->ticket;
    a.glob = sc->glob;
    a.resident_warps = (uint32_t)c->num_sms * (uint32_t)(CRYPT_THREADS / 32);

    int rc;
    if (c->flags & GIFT_CTX_CHECK_OVERLAP) {
        rc = launch_overlap_check(c, sc, a, st);
        if (rc != GIFT_OK) return rc;
        a.overlap = sc->overlap;
    }
    // Small tables take the fused form: one launch.  Every warp then checks the labels of the
    // segments it touches itself, so tables whose flat segments cover very many small units
    // stay with the split form, where that check runs once per segment.
    const bool cheap_labels = !labels || pages || MODE != MODE_ENCRYPT || labels->unit_bytes >= 256;
    if (allow_fused && nseg <= FUSED_MAX_SEGS && cheap_labels && !(c->flags & GIFT_CTX_SPLIT_LAUNCH)) {
        rc = launch_crypt<MODE>(c, a, st, true, true);
        if (rc != GIFT_OK) return rc;
    } else {
        const uint32_t plan_blocks = (nseg + 7) / 8;          // 8 warps per block, one warp per segment
        plan_kernel<MODE><<<plan_blocks, 256, 0, st>>>(a);
        scan_kernel<<<1, 1024, 0, st>>>(a);
        c->launches += 2;
        // Segments of one call do not overlap, so the buffer (or the page table) bounds their
        // average size; where that bound is small the pieces are short and the kernel that peels
        // their first row is the faster one.
        uint64_t room = buf_bytes;
        if (pages && (uint64_t)pages->n * pages->page_bytes < room) room = (uint64_t)pages->n * pages->page_bytes;
        rc = launch_crypt<MODE>(c, a, st, false, room / nseg <= SHORT_SEGMENT_BYTES);
        if (rc != GIFT_OK) return rc;
    }
    if (MODE == MODE_DECRYPT) {
        uint32_t fb = nseg < (uint32_t)c->num_sms * 8u ? nseg : (uint32_t)c->num_sms * 8u;
        fixup_kernel<<<fb, 256, 0, st>>>(a);
        c->launches++;
    }
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}

// Argument checks common to the three calls; GIFT_OK with *go == false means "nothing to do".
int seg_args_ok(gift_ctx* c, int mode, const void* src, void* dst, const gift_seg* segs, uint32_t nseg, uint32_t seg_base,
                const gift_pages* pages, const gift_labels* labels, const uint8_t* tags, const uint32_t* status, bool* go)
{
    *go = false;
    if (!c || !segs || !tags || !status) return nseg == 0 && c ? GIFT_OK : GIFT_E_INVAL;
    if (nseg == 0) return GIFT_OK;
    if (nseg > (1u << 30)) return GIFT_E_RANGE;
    if (!src || (mode != MODE_VERIFY && !dst)) return GIFT_E_INVAL;
    if (((uintptr_t)src & 15) || ((uintptr_t)dst & 15) || ((uintptr_t)tags & 15)) return GIFT_E_ALIGN;
    if (pages && (!pages->table || pages->page_bytes == 0)) return GIFT_E_INVAL;
    if (pages && (pages->page_bytes & 15)) return GIFT_E_ALIGN;
    if (labels && (!labels->owner_map || (!pages && labels->unit_bytes == 0))) return GIFT_E_INVAL;
    if (c->aad && (uint64_t)seg_base + nseg > c->aad_n) return GIFT_E_RANGE;      // more segments than bound AAD entries
    *go = true;
    return GIFT_OK;
}

}  // namespace

int gift_scratch_ensure(gift_ctx* c, SegScratch* sc, uint32_t nseg)
{
    if (nseg <= sc->cap) return GIFT_OK;
    uint32_t cap = sc->cap ? sc->cap : 1024u;
    while (cap < nseg) cap = cap > 0x7FFFFFFFu ? nseg : cap * 2u;
    CU_TRY(cudaDeviceSynchronize());
    Globals* glob = sc->glob;
    sc->glob = nullptr;
    gift_scratch_free(sc);
    sc->glob = glob;
    if (!sc->glob) {
        CU_TRY(cudaMalloc(&sc->glob, sizeof(Globals)));
        CU_TRY(cudaMemset(sc->glob, 0, sizeof(Globals)));
    }
    CU_TRY(cudaMalloc(&sc->wprefix, ((size_t)cap + 1) * sizeof(unsigned long long)));
    CU_TRY(cudaMalloc(&sc->acc, (size_t)cap * sizeof(uint4)));
    CU_TRY(cudaMalloc(&sc->ticket, (size_t)cap * sizeof(uint32_t)));
    CU_TRY(cudaMemset(sc->acc, 0, (size_t)cap * sizeof(uint4)));          // accumulators and tickets are zero between calls
    CU_TRY(cudaMemset(sc->ticket, 0, (size_t)cap * sizeof(uint32_t)));
    if (c->flags & GIFT_CTX_CHECK_OVERLAP) CU_TRY(cudaMalloc(&sc->overlap, cap));
    sc->cap = cap;
    return GIFT_OK;
}

void gift_scratch_free(SegScratch* sc)
{
    CU_NOTE(cudaFree(sc->wprefix));
    CU_NOTE(cudaFree(sc->acc));
    CU_NOTE(cudaFree(sc->ticket));
    CU_NOTE(cudaFree(sc->overlap));
    CU_NOTE(cudaFree(sc->glob));
    memset(sc, 0, sizeof(*sc));
}

int gift_seg_call_on(gift_ctx* c, int mode, SegScratch* sc, const void* src, void* dst, uint64_t buf_bytes,
                     const gift_seg* segs, uint32_t nseg, uint32_t seg_base, const gift_pages* pages,
                     const gift_labels* labels, uint8_t* tags, uint32_t* status, cudaStream_t st)
{
    bool go = false;
    int rc = seg_args_ok(c, mode, src, dst, segs, nseg, seg_base, pages, labels, tags, status, &go);
    if (rc != GIFT_OK || !go) return rc;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    rc = gift_scratch_ensure(c, sc, nseg);
    if (rc != GIFT_OK) return rc;
    switch (mode) {
    case MODE_ENCRYPT: return seg_call<MODE_ENCRYPT>(c, sc, src, dst, buf_bytes, segs, nseg, seg_base, pages, labels, tags, status, st, true);
    case MODE_DECRYPT: return seg_call<MODE_DECRYPT>(c, sc, src, dst, buf_bytes, segs, nseg, seg_base, pages, labels, tags, status, st, true);
    case MODE_VERIFY: return seg_call<MODE_VERIFY>(c, sc, src, dst, buf_bytes, segs, nseg, seg_base, pages, labels, tags, status, st, true);
    default: return GIFT_E_INVAL;
    }
}

// ---------------------------------------------------------------------------
// C entry points
// ---------------------------------------------------------------------------

extern "C" {

int gift_ctx_create(gift_ctx** out, int device, uint32_t max_users, uint32_t flags)
{
    if (!out || max_users == 0) return GIFT_E_INVAL;
    *out = nullptr;
    if (flags & ~(GIFT_CTX_TWO_TABLES | GIFT_CTX_CHECK_OVERLAP | GIFT_CTX_SPLIT_LAUNCH)) return GIFT_E_INVAL;
    if (max_users > (1u << 20)) return GIFT_E_RANGE;
    DeviceGuard g(device);
    if (!g.ok) return GIFT_E_CUDA;
    gift_ctx* c = new (std::nothrow) gift_ctx();
    if (!c) return GIFT_E_NOMEM;
    memset(c, 0, sizeof(*c));
    c->device = device;
    c->max_users = max_users;
    c->flags = flags;
    c->tables = (flags & GIFT_CTX_TWO_TABLES) ? 2 : 4;
    int rc = GIFT_OK;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete c; return GIFT_E_CUDA; }
    c->num_sms = prop.multiProcessorCount;
    auto fail = [&](int code) { gift_ctx_destroy(c); return code; };
    if (cudaMalloc(&c->d_t0, 256 * sizeof(uint32_t)) != cudaSuccess) return fail(GIFT_E_NOMEM);
    if (cudaMalloc(&c->d_isbox, 256) != cudaSuccess) return fail(GIFT_E_NOMEM);
    if (cudaMalloc(&c->d_hot, (size_t)max_users * sizeof(KeyHot)) != cudaSuccess) return fail(GIFT_E_NOMEM);
    if (cudaMalloc(&c->d_pow, (size_t)max_users * POW_LEVELS * 256 * sizeof(u128)) != cudaSuccess) return fail(GIFT_E_NOMEM);
    if (cudaMalloc(&c->d_rule_flags, (GIFT_CHAIN_MAX + 1) * sizeof(uint32_t)) != cudaSuccess) return fail(GIFT_E_NOMEM);
    if (cudaMemset(c->d_rule_flags, 0, (GIFT_CHAIN_MAX + 1) * sizeof(uint32_t)) != cudaSuccess) return fail(GIFT_E_CUDA);
    if (cudaMemset(c->d_hot, 0, (size_t)max_users * sizeof(KeyHot)) != cudaSuccess) return fail(GIFT_E_CUDA);
    if (cudaMemset(c->d_pow, 0, (size_t)max_users * POW_LEVELS * 256 * sizeof(u128)) != cudaSuccess) return fail(GIFT_E_CUDA);
    init_t0_kernel<<<1, 256>>>(c->d_t0, c->d_isbox);
    c->launches++;
    if (cudaDeviceSynchronize() != cudaSuccess) return fail(GIFT_E_CUDA);
    rc = gift_scratch_ensure(c, &c->scratch, 1024);
    if (rc != GIFT_OK) return fail(rc);
    const cudaError_t pending = cudaGetLastError();
    if (pending != cudaSuccess) {
        gift_note_cuda_error(pending, __FILE__, __LINE__);
        return fail(GIFT_E_CUDA);
    }
    *out = c;
    return GIFT_OK;
}

int gift_ctx_destroy(gift_ctx* c)
{
    if (!c) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (g.ok) {
        CU_NOTE(cudaDeviceSynchronize());
        if (c->d_hot) CU_NOTE(cudaMemset(c->d_hot, 0, (size_t)c->max_users * sizeof(KeyHot)));
        if (c->d_pow) CU_NOTE(cudaMemset(c->d_pow, 0, (size_t)c->max_users * POW_LEVELS * 256 * sizeof(u128)));
        if (c->d_stage_keys) CU_NOTE(cudaMemset(c->d_stage_keys, 0, (size_t)c->stage_cap * 16));
        CU_NOTE(cudaDeviceSynchronize());
        CU_NOTE(cudaFree(c->d_t0));
        CU_NOTE(cudaFree(c->d_isbox));
        CU_NOTE(cudaFree(c->d_hot));
        CU_NOTE(cudaFree(c->d_pow));
        gift_scratch_free(&c->scratch);
        CU_NOTE(cudaFree(c->d_claim));
        CU_NOTE(cudaFree(c->d_rule_flags));
        if (c->io_ready) {
            for (int i = 0; i < GIFT_IO_STREAMS; i++) {
                gift_scratch_free(&c->io_scratch[i]);
                if (c->io_done[i]) CU_NOTE(cudaEventDestroy(c->io_done[i]));
                if (c->io_stream[i]) CU_NOTE(cudaStreamDestroy(c->io_stream[i]));
            }
            if (c->io_start) CU_NOTE(cudaEventDestroy(c->io_start));
        }
        CU_NOTE(cudaFree(c->d_stage_ids));
        CU_NOTE(cudaFree(c->d_stage_keys));
        CU_NOTE(cudaFree(c->d_snapshot));
        CU_NOTE(cudaFree(c->d_next_sync));
        if (c->h_stage) {
            memset(c->h_stage, 0, (size_t)c->stage_cap * 20);
            CU_NOTE(cudaFreeHost(c->h_stage));
        }
        if (c->ev) {
            for (uint32_t i = 0; i < 2 * MAX_TIMED; i++) CU_NOTE(cudaEventDestroy(c->ev[i]));
            delete[] c->ev;
        }
        CU_NOTE(cudaGetLastError());
    }
    delete c;
    return GIFT_OK;
}

int gift_ctx_reserve(gift_ctx* c, uint32_t max_segs)
{
    if (!c) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    return gift_scratch_ensure(c, &c->scratch, max_segs);
}

static int stage_ids(gift_ctx* c, const int32_t* user_ids, const uint8_t* keys16, uint32_t n, cudaStream_t st)
{
    for (uint32_t i = 0; i < n; i++)
        if (user_ids[i] < 0 || (uint32_t)user_ids[i] >= c->max_users) return GIFT_E_RANGE;
    if (n > c->stage_cap) {
        CU_TRY(cudaDeviceSynchronize());
        if (c->h_stage) { memset(c->h_stage, 0, (size_t)c->stage_cap * 20); cudaFreeHost(c->h_stage); c->h_stage = nullptr; }
        cudaFree(c->d_stage_ids); cudaFree(c->d_stage_keys);
        c->d_stage_ids = nullptr; c->d_stage_keys = nullptr; c->stage_cap = 0;
        CU_TRY(cudaMallocHost(&c->h_stage, (size_t)n * 20));
        CU_TRY(cudaMalloc(&c->d_stage_ids, (size_t)n * 4));
        CU_TRY(cudaMalloc(&c->d_stage_keys, (size_t)n * 16));
        c->stage_cap = n;
    } else {
        // the staging buffers may still be in use by an earlier call on another stream
        CU_TRY(cudaDeviceSynchronize());
    }
    memcpy(c->h_stage, user_ids, (size_t)n * 4);
    CU_TRY(cudaMemcpyAsync(c->d_stage_ids, c->h_stage, (size_t)n * 4, cudaMemcpyHostToDevice, st));
    if (keys16) {
        memcpy(c->h_stage + (size_t)n * 4, keys16, (size_t)n * 16);
        CU_TRY(cudaMemcpyAsync(c->d_stage_keys, c->h_stage + (size_t)n * 4, (size_t)n * 16, cudaMemcpyHostToDevice, st));
    }
    return GIFT_OK;
}

int gift_set_keys(gift_ctx* c, const int32_t* user_ids, const uint8_t* keys16, uint32_t n, void* stream)
{
    if (!c || (n && (!user_ids || !keys16))) return GIFT_E_INVAL;
    if (n == 0) return GIFT_OK;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = stage_ids(c, user_ids, keys16, n, st);
    if (rc != GIFT_OK) return rc;
    const uint32_t threads = n * POW_LEVELS;
    key_setup_kernel<<<(threads + 63) / 64, 64, 0, st>>>(c->d_t0, c->d_stage_ids, c->d_stage_keys, n, c->d_hot, c->d_pow);
    c->launches++;
    // wipe the staging copies once the kernel has consumed them
    CU_TRY(cudaMemsetAsync(c->d_stage_keys, 0, (size_t)n * 16, st));
    CU_TRY(cudaStreamSynchronize(st));
    memset(c->h_stage, 0, (size_t)n * 20);
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}

int gift_clear_keys(gift_ctx* c, const int32_t* user_ids, uint32_t n, void* stream)
{
    if (!c || (n && !user_ids)) return GIFT_E_INVAL;
    if (n == 0) return GIFT_OK;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = stage_ids(c, user_ids, nullptr, n, st);
    if (rc != GIFT_OK) return rc;
    key_clear_kernel<<<n, 256, 0, st>>>(c->d_stage_ids, n, c->d_hot, c->d_pow);
    c->launches++;
    CU_TRY(cudaStreamSynchronize(st));
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}

int gift_seg_encrypt(gift_ctx* c, const void* src, void* dst, uint64_t buf_bytes, const gift_seg* segs,
                     uint32_t nseg, const gift_pages* pages, const gift_labels* labels, uint8_t* tags_out,
                     uint32_t* status, void* stream)
{
    return gift_seg_call_on(c, MODE_ENCRYPT, c ? &c->scratch : nullptr, src, dst, buf_bytes, segs, nseg, 0, pages, labels,
                            tags_out, status, (cudaStream_t)stream);
}

int gift_seg_decrypt(gift_ctx* c, const void* src, void* dst, uint64_t buf_bytes, const gift_seg* segs,
                     uint32_t nseg, const gift_pages* pages, gift_labels* labels, const uint8_t* tags_in,
                     uint32_t* status, void* stream)
{
    return gift_seg_call_on(c, MODE_DECRYPT, c ? &c->scratch : nullptr, src, dst, buf_bytes, segs, nseg, 0, pages, labels,
                            (uint8_t*)tags_in, status, (cudaStream_t)stream);
}

int gift_verify_tags(gift_ctx* c, const void* src, uint64_t buf_bytes, const gift_seg* segs, uint32_t nseg,
                     const gift_pages* pages, const uint8_t* tags_in, uint32_t* status, void* stream)
{
    return gift_seg_call_on(c, MODE_VERIFY, c ? &c->scratch : nullptr, src, nullptr, buf_bytes, segs, nseg, 0, pages, nullptr,
                            (uint8_t*)tags_in, status, (cudaStream_t)stream);
}

int gift_ctx_bind_aad(gift_ctx* c, const uint8_t* aad16, uint32_t n)
{
    if (!c) return GIFT_E_INVAL;
    if ((uintptr_t)aad16 & 15) return GIFT_E_ALIGN;
    c->aad = aad16;
    c->aad_n = aad16 ? n : 0;
    return GIFT_OK;
}

int gift_timing_enable(gift_ctx* c, int on)
{
    if (!c) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    if (on && !c->ev) {
        c->ev = new (std::nothrow) cudaEvent_t[2 * MAX_TIMED];
        if (!c->ev) return GIFT_E_NOMEM;
        for (uint32_t i = 0; i < 2 * MAX_TIMED; i++) {
            if (cudaEventCreate(&c->ev[i]) != cudaSuccess) {
                for (uint32_t k = 0; k < i; k++) cudaEventDestroy(c->ev[k]);
                delete[] c->ev;
                c->ev = nullptr;
                return GIFT_E_CUDA;
            }
        }
    }
    c->timing = on ? 1 : 0;
    c->n_timed = 0;
    return GIFT_OK;
}

int gift_timing_read(gift_ctx* c, double* total_ms, uint32_t* launches)
{
    if (!c || !total_ms || !launches) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    double sum = 0.0;
    for (uint32_t i = 0; i < c->n_timed; i++) {
        float ms = 0.f;
        CU_TRY(cudaEventSynchronize(c->ev[2 * i + 1]));
        CU_TRY(cudaEventElapsedTime(&ms, c->ev[2 * i], c->ev[2 * i + 1]));
        sum += ms;
    }
    *total_ms = sum;
    *launches = c->n_timed;
    c->n_timed = 0;
    return GIFT_OK;
}

const char* gift_strerror(int code)
{
    switch (code) {
    case GIFT_OK: return "ok";
    case GIFT_E_INVAL: return "invalid argument";
    case GIFT_E_NOMEM: return "out of memory";
    case GIFT_E_CUDA: return "CUDA runtime error";
    case GIFT_E_RANGE: return "value out of range";
    case GIFT_E_ALIGN: return "pointer or size not 16-byte aligned";
    default: return "unknown error";
    }
}

const char* gift_last_error_detail(void) { return g_error_detail; }

uint32_t gift_version(void) { return GIFT_VERSION; }

uint64_t gift_launch_count(const gift_ctx* c) { return c ? c->launches : 0; }

}  // extern "C"

// ---------------------------------------------------------------------------
// gift_seg_encrypt_static: the export call for callers that must not allocate
// ---------------------------------------------------------------------------
//
// Same kernels as gift_seg_encrypt (always the split form, whose plan kernel clears what a
// call needs), but the per-call scratch (work list, partial hashes, tickets, counters) lives
// in one file-scope device array instead of memory the ctx grows with cudaMalloc.  The
// array belongs to the loaded library: every GPU that loads libgift.so holds
// STATIC_SCRATCH_BYTES of it until the process exits, and every call on that GPU shares it.

namespace {

constexpr size_t STATIC_OFF_PREFIX = 256;                                                   // after Globals
constexpr size_t STATIC_OFF_ACC = STATIC_OFF_PREFIX + ((size_t)GIFT_STATIC_MAX_SEGS + 64) * 8;   // 16-byte aligned
constexpr size_t STATIC_OFF_TICKET = STATIC_OFF_ACC + (size_t)GIFT_STATIC_MAX_SEGS * 16;
constexpr size_t STATIC_OFF_OVERLAP = STATIC_OFF_TICKET + (size_t)GIFT_STATIC_MAX_SEGS * 4;
constexpr size_t STATIC_SCRATCH_BYTES = STATIC_OFF_OVERLAP + (size_t)GIFT_STATIC_MAX_SEGS;
static_assert(sizeof(Globals) <= STATIC_OFF_PREFIX && STATIC_OFF_ACC % 16 == 0, "static scratch layout");

// In host code this name is only a handle for the symbol, never a device address:
// the address a kernel can use comes from cudaGetSymbolAddress, per device.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int STATIC_MAX_DEVICES = 64;
unsigned char* g_static_ptr[STATIC_MAX_DEVICES];      // device address of the array on each GPU, once known

// First use on a device: look the symbol up with that device current.
int static_scratch_for(int device, unsigned char** out)
{
    if (device < 0 || device >= STATIC_MAX_DEVICES) return GIFT_E_RANGE;
    if (g_static_ptr[device] == nullptr) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || p == nullptr) return GIFT_E_CUDA;
        g_static_ptr[device] = static_cast<unsigned char*>(p);
    }
    *out = g_static_ptr[device];
    return GIFT_OK;
}

}  // namespace

extern "C" int gift_seg_encrypt_static(gift_ctx* c, const void* src, void* dst, uint64_t buf_bytes,
                                       const gift_seg* segs, uint32_t nseg, const gift_pages* pages,
                                       const gift_labels* labels, uint8_t* tags_out, uint32_t* status,
                                       void* stream)
{
    if (c && nseg > GIFT_STATIC_MAX_SEGS) return GIFT_E_RANGE;     // larger tables need gift_seg_encrypt
    bool go = false;
    int rc = seg_args_ok(c, MODE_ENCRYPT, src, dst, segs, nseg, 0, pages, labels, tags_out, status, &go);
    if (rc != GIFT_OK || !go) return rc;
    // the overlap check of paged tables keeps a claim array that grows with cudaMalloc
    if ((c->flags & GIFT_CTX_CHECK_OVERLAP) && pages) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    unsigned char* scratch = nullptr;
    rc = static_scratch_for(c->device, &scratch);
    if (rc != GIFT_OK) return rc;
    SegScratch sc;
    sc.cap = GIFT_STATIC_MAX_SEGS;
    sc.glob = reinterpret_cast<Globals*>(scratch);
    sc.wprefix = reinterpret_cast<unsigned long long*>(scratch + STATIC_OFF_PREFIX);
    sc.acc = reinterpret_cast<uint4*>(scratch + STATIC_OFF_ACC);
    sc.ticket = reinterpret_cast<uint32_t*>(scratch + STATIC_OFF_TICKET);
    sc.overlap = scratch + STATIC_OFF_OVERLAP;
    // The array still holds the previous call's values: the per-segment accumulators and tickets
    // are cleared by the plan kernel, the weight prefix and the counters are rewritten by the
    // scan kernel before the cipher kernel reads them.
    return seg_call<MODE_ENCRYPT>(c, &sc, src, dst, buf_bytes, segs, nseg, 0, pages, labels, tags_out, status,
                                  (cudaStream_t)stream, false);
}
