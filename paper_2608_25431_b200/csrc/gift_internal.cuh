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

struct gift_ctx {
    int device;
    uint32_t max_users;
    uint32_t flags;
    int chains;                        // Horner chains per lane (1 or 2)
    int tables;                        // T-tables held in shared memory (2 or 4)
    int threads;                       // threads per CTA of the cipher kernel (512, 768 or 1024)
    int num_sms;
    uint32_t* d_t0;                    // 256-entry T0 in global memory
    uint8_t* d_isbox;                  // 256-entry inverse S-box (token mode)
    gift::KeyHot* d_hot;                     // [max_users]
    gift::u128* d_pow;                       // [max_users][POW_LEVELS*256]
    uint8_t* h_stage;                  // pinned staging for keys
    uint32_t stage_cap;                // users the staging buffers hold
    int32_t* d_stage_ids;
    uint8_t* d_stage_keys;
    uint32_t seg_cap;
    unsigned long long* d_wprefix;     // [seg_cap + 1] exclusive prefix of the segment weights
    uint4* d_acc;                      // [seg_cap]
    uint32_t* d_ticket;                // [seg_cap]
    Globals* d_glob;
    int32_t* d_next_sync;              // launch-order check: completion time per launch
    uint32_t order_cap;
    int32_t* d_snapshot;               // label snapshot for aliased rules
    uint32_t snapshot_cap;
    const uint8_t* aad;                // per-segment additional authenticated data bound to the next calls, or nullptr
    uint64_t launches;
    int timing;                        // record events around the cipher kernel
    uint32_t n_timed;
    cudaEvent_t* ev;                   // 2 * MAX_TIMED events, created on first enable
};

#define MAX_TIMED 1024u

#define CU_TRY(expr)                                   \
    do {                                               \
        cudaError_t e_ = (expr);                       \
        if (e_ != cudaSuccess) {                       \
            return e_ == cudaErrorMemoryAllocation ? GIFT_E_NOMEM : GIFT_E_CUDA; \
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

