// Internal definitions shared by the translation units of libgift: the context, the
// per-call counters, error mapping and the device guard.  Not part of the public ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/gift.h"
#include "gift_core.cuh"

// ---------------------------------------------------------------------------
// context
// ---------------------------------------------------------------------------

struct Globals {
    unsigned long long total_weight;   // sum of the accepted segments' weights (see scan_kernel)
    unsigned long long slice;          // weight handed to each resident warp
    uint32_t pad[4];
};

// Per-call scratch of the segment kernels.  One set serves one stream at a time; the ctx has
// one for the plain calls and one per internal stream of the host-boundary calls.  The hash
// accumulators and tickets are zero between calls (cleared at allocation, and by the warp that
// finishes a segment).
struct SegScratch {
    uint32_t cap;                      // segments the arrays hold
    unsigned long long* wprefix;       // [cap + 1] exclusive prefix of the segment weights
    uint4* acc;                        // [cap]
    uint32_t* ticket;                  // [cap]
    uint8_t* overlap;                  // [cap] overlap flags (only with GIFT_CTX_CHECK_OVERLAP)
    Globals* glob;
};

#define GIFT_IO_STREAMS 3

struct gift_ctx {
    int device;
    uint32_t max_users;
    uint32_t flags;
    int tables;                        // T-tables held in shared memory (2 or 4)
    int num_sms;
    uint32_t* d_t0;                    // 256-entry T0 in global memory
    uint8_t* d_isbox;                  // 256-entry inverse S-box (token mode)
    gift::KeyHot* d_hot;                     // [max_users]
    gift::u128* d_pow;                       // [max_users][POW_LEVELS*256]
    uint8_t* h_stage;                  // pinned staging for keys
    uint32_t stage_cap;                // users the staging buffers hold
    int32_t* d_stage_ids;
    uint8_t* d_stage_keys;
    SegScratch scratch;                // plain calls
    int32_t* d_claim;                  // overlap check, paged mode: first claimant of every physical page
    uint64_t claim_cap;
    // host-boundary calls (gift_export_to_host / gift_import_from_host), created on first use
    cudaStream_t io_stream[GIFT_IO_STREAMS];
    cudaEvent_t io_done[GIFT_IO_STREAMS];
    cudaEvent_t io_start;
    SegScratch io_scratch[GIFT_IO_STREAMS];
    int io_ready;
    uint32_t io_next;                  // internal stream the next chunk goes to
    int32_t* d_next_sync;              // launch-order check: completion time per launch
    uint32_t order_cap;
    int32_t* d_snapshot;               // label snapshot for aliased rules
    uint32_t* d_rule_flags;            // [GIFT_CHAIN_MAX] 1: the rule's index arrays are malformed
    uint32_t snapshot_cap;
    const uint8_t* aad;                // per-segment additional authenticated data bound to the next calls, or nullptr
    uint32_t aad_n;                    // entries of the bound array
    uint64_t launches;
    int timing;                        // record events around the cipher kernel
    uint32_t n_timed;
    cudaEvent_t* ev;                   // 2 * MAX_TIMED events, created on first enable
};

// One segment call (mode: gift::MODE_*) on `st` with the given scratch set; the arguments of
// gift_seg_encrypt / decrypt / verify after validation.  seg_base is the index of segs[0] in
// the caller's whole table (the bound AAD array is indexed from there).
int gift_seg_call_on(gift_ctx* c, int mode, SegScratch* sc, const void* src, void* dst, uint64_t buf_bytes,
                     const gift_seg* segs, uint32_t nseg, uint32_t seg_base, const gift_pages* pages,
                     const gift_labels* labels, uint8_t* tags, uint32_t* status, cudaStream_t st);
int gift_scratch_ensure(gift_ctx* c, SegScratch* sc, uint32_t nseg);
void gift_scratch_free(SegScratch* sc);

#define MAX_TIMED 1024u

// Where the last failing CUDA runtime call of this thread was, for gift_last_error_detail().
void gift_note_cuda_error(cudaError_t e, const char* file, int line);

#define CU_TRY(expr)                                   \
    do {                                               \
        cudaError_t e_ = (expr);                       \
        if (e_ != cudaSuccess) {                       \
            gift_note_cuda_error(e_, __FILE__, __LINE__); \
            return e_ == cudaErrorMemoryAllocation ? GIFT_E_NOMEM : GIFT_E_CUDA; \
        }                                              \
    } while (0)


// For clean-up paths that go on regardless: remember a failure, clear it, continue.
#define CU_NOTE(expr)                                  \
    do {                                               \
        cudaError_t e_ = (expr);                       \
        if (e_ != cudaSuccess) {                       \
            gift_note_cuda_error(e_, __FILE__, __LINE__); \
            (void)cudaGetLastError();                  \
        }                                              \
    } while (0)

// Makes a device current for the duration of a call and restores the previous one.
struct DeviceGuard {
    int prev;
    bool ok;
    explicit DeviceGuard(int dev) : prev(-1), ok(false)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = prev == dev || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard()
    {
        if (ok && prev >= 0) cudaSetDevice(prev);
    }
};

