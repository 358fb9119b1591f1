// Host-boundary calls: export to and import from page-locked host memory with the copies
// fused into the call (paper sec. 4.5, the swap path of KV blocks; sec. 5, the bounce copy).
//
// A caller whose data crosses the CPU/GPU boundary needs copy + cipher + copy.  Done in one
// piece the three stages run back to back and the bus idles while the cipher runs and the
// other way round.  Here the table is cut into chunks that no segment straddles; chunk k
// goes to internal stream k mod 3 of the ctx, each with its own scratch set, so that the
// upload of one chunk, the cipher of the previous one and the download of the one before
// overlap.  Export is out of place into a cleared staging range, so that nothing but
// ciphertext and zeros can reach the host side: a segment the label check refuses stays
// plaintext on the device and arrives as zeros.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "gift_internal.cuh"

using namespace gift;

namespace {

int io_init(gift_ctx* c)
{
    if (c->io_ready) return GIFT_OK;
    for (int i = 0; i < GIFT_IO_STREAMS; i++) {
        CU_TRY(cudaStreamCreateWithFlags(&c->io_stream[i], cudaStreamNonBlocking));
        CU_TRY(cudaEventCreateWithFlags(&c->io_done[i], cudaEventDisableTiming));
    }
    CU_TRY(cudaEventCreateWithFlags(&c->io_start, cudaEventDisableTiming));
    c->io_ready = 1;
    return GIFT_OK;
}

int chunks_ok(const gift_chunk* chunks, uint32_t n_chunks, uint64_t buf_bytes, uint32_t nseg)
{
    if (n_chunks && !chunks) return GIFT_E_INVAL;
    for (uint32_t k = 0; k < n_chunks; k++) {
        const gift_chunk& ch = chunks[k];
        if (ch.seg_lo > ch.seg_hi || ch.seg_hi > nseg) return GIFT_E_INVAL;
        if (ch.byte_lo > ch.byte_hi || ch.byte_hi > buf_bytes) return GIFT_E_INVAL;
        if ((ch.byte_lo & 15) || (ch.byte_hi & 15)) return GIFT_E_ALIGN;
    }
    return GIFT_OK;
}

// Scratch for the largest chunk on every internal stream, before anything is enqueued
// (growing scratch synchronises the device).
int io_reserve(gift_ctx* c, const gift_chunk* chunks, uint32_t n_chunks)
{
    uint32_t most = 1;
    for (uint32_t k = 0; k < n_chunks; k++)
        if (chunks[k].seg_hi - chunks[k].seg_lo > most) most = chunks[k].seg_hi - chunks[k].seg_lo;
    for (int i = 0; i < GIFT_IO_STREAMS; i++) {
        const int rc = gift_scratch_ensure(c, &c->io_scratch[i], most);
        if (rc != GIFT_OK) return rc;
    }
    return GIFT_OK;
}

// The internal stream the next chunk goes to, made to wait for the caller's stream the first
// time the call uses it.  With the overlap check of paged tables there is one claim array per
// ctx, so every chunk then goes to the same stream.
int io_slot(gift_ctx* c, bool used[GIFT_IO_STREAMS])
{
    const int slot = (c->flags & GIFT_CTX_CHECK_OVERLAP) ? 0 : (int)(c->io_next++ % GIFT_IO_STREAMS);
    if (!used[slot]) {
        if (cudaStreamWaitEvent(c->io_stream[slot], c->io_start, 0) != cudaSuccess) return -1;
        used[slot] = true;
    }
    return slot;
}

// The caller's stream waits for every internal stream the call used.
int io_join(gift_ctx* c, const bool used[GIFT_IO_STREAMS], cudaStream_t user)
{
    for (int i = 0; i < GIFT_IO_STREAMS; i++) {
        if (!used[i]) continue;
        CU_TRY(cudaEventRecord(c->io_done[i], c->io_stream[i]));
        CU_TRY(cudaStreamWaitEvent(user, c->io_done[i], 0));
    }
    return GIFT_OK;
}

}  // namespace

extern "C" int gift_export_to_host(gift_ctx* c, const void* h_src, void* h_dst, void* d_plain, void* d_cipher,
                                   uint64_t buf_bytes, const gift_seg* segs, uint32_t nseg, const gift_chunk* chunks,
                                   uint32_t n_chunks, const gift_pages* pages, const gift_labels* labels,
                                   uint8_t* d_tags, uint32_t* d_status, uint8_t* h_tags, uint32_t* h_status,
                                   void* stream)
{
    if (!c) return GIFT_E_INVAL;
    if (n_chunks == 0) return GIFT_OK;
    if (!h_dst || !d_plain || !d_cipher || d_plain == d_cipher) return GIFT_E_INVAL;
    if (nseg && (!segs || !d_tags || !d_status || !h_tags || !h_status)) return GIFT_E_INVAL;
    int rc = chunks_ok(chunks, n_chunks, buf_bytes, nseg);
    if (rc != GIFT_OK) return rc;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    rc = io_init(c);
    if (rc != GIFT_OK) return rc;
    rc = io_reserve(c, chunks, n_chunks);
    if (rc != GIFT_OK) return rc;
    cudaStream_t user = (cudaStream_t)stream;
    CU_TRY(cudaEventRecord(c->io_start, user));
    bool used[GIFT_IO_STREAMS] = {false, false, false};
    // one chunk: upload, clear, encrypt out of place, download
    auto enqueue = [&](const gift_chunk& ch) -> int {
        const int slot = io_slot(c, used);
        if (slot < 0) return GIFT_E_CUDA;
        cudaStream_t st = c->io_stream[slot];
        const uint64_t nb = ch.byte_hi - ch.byte_lo;
        const uint32_t ns = ch.seg_hi - ch.seg_lo;
        uint8_t* plain = (uint8_t*)d_plain + ch.byte_lo;
        uint8_t* cipher = (uint8_t*)d_cipher + ch.byte_lo;
        if (nb) {
            if (h_src) CU_TRY(cudaMemcpyAsync(plain, (const uint8_t*)h_src + ch.byte_lo, nb, cudaMemcpyHostToDevice, st));
            CU_TRY(cudaMemsetAsync(cipher, 0, nb, st));
        }
        if (ns) {
            const int rc2 = gift_seg_call_on(c, MODE_ENCRYPT, &c->io_scratch[slot], d_plain, d_cipher, buf_bytes, segs + ch.seg_lo,
                                             ns, ch.seg_lo, pages, labels, d_tags + 16 * (size_t)ch.seg_lo, d_status + ch.seg_lo, st);
            if (rc2 != GIFT_OK) return rc2;
        }
        if (nb) CU_TRY(cudaMemcpyAsync((uint8_t*)h_dst + ch.byte_lo, cipher, nb, cudaMemcpyDeviceToHost, st));
        if (ns) {
            CU_TRY(cudaMemcpyAsync(h_tags + 16 * (size_t)ch.seg_lo, d_tags + 16 * (size_t)ch.seg_lo, (size_t)ns * 16,
                                   cudaMemcpyDeviceToHost, st));
            CU_TRY(cudaMemcpyAsync(h_status + ch.seg_lo, d_status + ch.seg_lo, (size_t)ns * 4, cudaMemcpyDeviceToHost, st));
        }
        return GIFT_OK;
    };
    rc = GIFT_OK;
    for (uint32_t k = 0; k < n_chunks && rc == GIFT_OK; k++) rc = enqueue(chunks[k]);
    const int rc_join = io_join(c, used, user);       // also after a failure: what was enqueued must not outrun the caller's stream
    return rc != GIFT_OK ? rc : rc_join;
}

extern "C" int gift_import_from_host(gift_ctx* c, const void* h_src, const uint8_t* h_tags, void* d_buf,
                                     uint64_t buf_bytes, const gift_seg* segs, uint32_t nseg, const gift_chunk* chunks,
                                     uint32_t n_chunks, const gift_pages* pages, gift_labels* labels, uint8_t* d_tags,
                                     uint32_t* d_status, uint32_t* h_status, void* stream)
{
    if (!c) return GIFT_E_INVAL;
    if (n_chunks == 0) return GIFT_OK;
    if (!h_src || !d_buf) return GIFT_E_INVAL;
    if (nseg && (!segs || !d_tags || !d_status || !h_tags || !h_status)) return GIFT_E_INVAL;
    int rc = chunks_ok(chunks, n_chunks, buf_bytes, nseg);
    if (rc != GIFT_OK) return rc;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    rc = io_init(c);
    if (rc != GIFT_OK) return rc;
    rc = io_reserve(c, chunks, n_chunks);
    if (rc != GIFT_OK) return rc;
    cudaStream_t user = (cudaStream_t)stream;
    CU_TRY(cudaEventRecord(c->io_start, user));
    bool used[GIFT_IO_STREAMS] = {false, false, false};
    // one chunk: upload ciphertext and tags, decrypt in place, status words back
    auto enqueue = [&](const gift_chunk& ch) -> int {
        const int slot = io_slot(c, used);
        if (slot < 0) return GIFT_E_CUDA;
        cudaStream_t st = c->io_stream[slot];
        const uint64_t nb = ch.byte_hi - ch.byte_lo;
        const uint32_t ns = ch.seg_hi - ch.seg_lo;
        if (nb) CU_TRY(cudaMemcpyAsync((uint8_t*)d_buf + ch.byte_lo, (const uint8_t*)h_src + ch.byte_lo, nb, cudaMemcpyHostToDevice, st));
        if (ns) {
            CU_TRY(cudaMemcpyAsync(d_tags + 16 * (size_t)ch.seg_lo, h_tags + 16 * (size_t)ch.seg_lo, (size_t)ns * 16,
                                   cudaMemcpyHostToDevice, st));
            const int rc2 = gift_seg_call_on(c, MODE_DECRYPT, &c->io_scratch[slot], d_buf, d_buf, buf_bytes, segs + ch.seg_lo, ns,
                                             ch.seg_lo, pages, labels, d_tags + 16 * (size_t)ch.seg_lo, d_status + ch.seg_lo, st);
            if (rc2 != GIFT_OK) return rc2;
            CU_TRY(cudaMemcpyAsync(h_status + ch.seg_lo, d_status + ch.seg_lo, (size_t)ns * 4, cudaMemcpyDeviceToHost, st));
        }
        return GIFT_OK;
    };
    rc = GIFT_OK;
    for (uint32_t k = 0; k < n_chunks && rc == GIFT_OK; k++) rc = enqueue(chunks[k]);
    const int rc_join = io_join(c, used, user);
    return rc != GIFT_OK ? rc : rc_join;
}
