// Device side of gift_seg_encrypt / gift_seg_decrypt / gift_verify_tags.
//
// A call runs, on the caller's stream and with no host round trip in between, either
//
//   the split form (any table size)
//     1. plan_kernel     one warp per segment: descriptor checks, ownership-label check,
//                        pre-status, cleared hash accumulators, the segment's weight
//     2. scan_kernel     prefix sum of the weights and the weight slice of a resident warp
//     3. crypt_kernel    every resident warp takes its slice; per piece of a segment: CTR
//                        keystream + XOR + GHASH; the warp whose report completes a segment
//                        finishes its tag (no waiting, tickets only)
//   or the fused form (tables of at most FUSED_MAX_SEGS segments: the rows of a decode step)
//     1. crypt_kernel<FUSED>  every CTA reads the table into shared memory and recomputes the
//                        weights and their prefix sum there (a microsecond of redundant
//                        work instead of three kernel boundaries); every warp checks the
//                        segments its slice touches itself
//   followed, for decrypt, by
//     4. fixup_kernel    zero-fills failed segments and marks their units unowned.
//
// AES uses T-tables replicated across the 32 shared-memory banks so that a warp's 32
// data-dependent lookups never conflict; GHASH uses masked integer multiplies (gf128.cuh).
// The path is bound by the integer pipes, not by HBM: about one eighth of the memory
// bandwidth is needed, so data moves with plain 128-bit loads and stores and no staging
// through shared memory.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/gift.h"
#include "gift_core.cuh"
#include "gift_internal.cuh"

namespace gift {

// ---------------------------------------------------------------------------
// call parameters shared by the segment kernels
// ---------------------------------------------------------------------------

struct CallArgs {
    const uint8_t* src;
    uint8_t* dst;
    uint64_t buf_bytes;
    const gift_seg* segs;
    uint32_t nseg;
    const int32_t* page_table;     // nullptr: flat
    uint32_t n_pages;
    uint64_t page_bytes;
    int32_t* owner_map;            // nullptr: no labels
    uint32_t n_units;
    uint64_t unit_bytes;
    uint8_t* tags;                 // out (encrypt) or in (decrypt, verify)
    const uint8_t* aad;            // 16 bytes of additional authenticated data per segment, or nullptr
    uint32_t* status;
    const KeyHot* hot;
    const u128* pow;
    uint32_t max_users;
    unsigned long long* wprefix;   // [nseg + 1] exclusive prefix of the segment weights (split form)
    uint4* acc;                    // [nseg] combined hash of segments cut into several pieces; zero between calls
    uint32_t* ticket;              // [nseg] pieces that have reported; zero between calls
    Globals* glob;
    const uint8_t* overlap;        // [nseg] 1: the segment shares bytes with another one (overlap check on), or nullptr
    uint32_t resident_warps;       // warps of the cipher kernel on the whole GPU
};

constexpr int CRYPT_THREADS = 768;           // 24 warps per SM at 80 registers per thread
constexpr uint32_t FUSED_MAX_SEGS = 1024;    // largest table the fused form takes

__device__ __forceinline__ uint64_t seg_blocks(uint64_t len) { return (len + 15) >> 4; }

// Units a segment covers: flat, [u0, u0 + count); paged, one per page.
__device__ __forceinline__ uint64_t seg_unit_count(const CallArgs& a, const gift_seg& s, uint64_t* u0)
{
    if (s.len == 0) { *u0 = 0; return 0; }
    if (a.page_table == nullptr) {
        *u0 = s.offset / a.unit_bytes;
        const uint64_t u1 = (s.offset + s.len + a.unit_bytes - 1) / a.unit_bytes;
        return u1 - *u0;
    }
    *u0 = 0;
    return (s.len + a.page_bytes - 1) / a.page_bytes;
}

__device__ __forceinline__ uint64_t seg_unit(const CallArgs& a, const gift_seg& s, uint64_t u0, uint64_t k)
{
    if (a.page_table == nullptr) return u0 + k;
    return (uint64_t)(uint32_t)a.page_table[(uint64_t)s.page0 + k];
}

// ---------------------------------------------------------------------------
// descriptor and label checks (paper sec. 3 step 4, sec. 4.2)
// ---------------------------------------------------------------------------

// The part of the descriptor check that needs no table walk; one thread.
__device__ __forceinline__ bool desc_bad_quick(const CallArgs& a, const gift_seg& seg)
{
    if (seg.flags != 0 || seg.len > GIFT_MAX_SEG_BYTES) return true;
    if (a.page_table == nullptr) {
        if ((seg.offset & 15) != 0 || seg.offset > a.buf_bytes || seg.len > a.buf_bytes - seg.offset) return true;
        if (a.owner_map != nullptr && seg.len > 0) {
            const uint64_t u1 = (seg.offset + seg.len + a.unit_bytes - 1) / a.unit_bytes;
            if (u1 > a.n_units) return true;
        }
        return false;
    }
    const uint64_t np = (seg.len + a.page_bytes - 1) / a.page_bytes;
    return (uint64_t)seg.page0 + np > a.n_pages;
}

// Status of one segment before any byte of it is touched, computed by a whole warp (every
// lane returns the same word): BAD_DESC alone, or OVERLAP alone, or any of UNOWNED,
// OWNER_MISMATCH (encrypt with labels) and NO_KEY.
template <int MODE>
__device__ __forceinline__ uint32_t seg_prestatus(const CallArgs& a, const gift_seg& seg, uint32_t s, int lane)
{
    const bool labels = a.owner_map != nullptr;
    bool bad = desc_bad_quick(a, seg);
    if (!bad && a.page_table != nullptr) {
        const uint64_t np = (seg.len + a.page_bytes - 1) / a.page_bytes;
        bool b = false;
        for (uint64_t k = lane; k < np; k += 32) {
            const int32_t t = a.page_table[(uint64_t)seg.page0 + k];
            b |= t < 0 || ((uint64_t)t + 1) * a.page_bytes > a.buf_bytes || (labels && (uint64_t)t >= a.n_units);
        }
        bad = __any_sync(0xFFFFFFFFu, b);
    }
    if (bad) return GIFT_ST_BAD_DESC;
    if (a.overlap != nullptr && a.overlap[s] != 0) return GIFT_ST_OVERLAP;
    uint32_t st = 0;
    if (MODE == MODE_ENCRYPT && labels) {
        uint64_t u0;
        const uint64_t nu = seg_unit_count(a, seg, &u0);
        bool unowned = false, mism = false;
        for (uint64_t k = lane; k < nu; k += 32) {
            const int32_t l = a.owner_map[seg_unit(a, seg, u0, k)];
            unowned |= l <= GIFT_OWNER_NONE;
            mism |= l == GIFT_OWNER_PARAM || (l >= 0 && l != seg.owner);
        }
        if (__any_sync(0xFFFFFFFFu, unowned)) st |= GIFT_ST_UNOWNED;
        if (__any_sync(0xFFFFFFFFu, mism)) st |= GIFT_ST_OWNER_MISMATCH;
    }
    const bool has_key = seg.owner >= 0 && (uint32_t)seg.owner < a.max_users && a.hot[seg.owner].valid != 0;
    if (!has_key) st |= GIFT_ST_NO_KEY;
    return st;
}

// ---------------------------------------------------------------------------
// 1. plan (split form)
// ---------------------------------------------------------------------------

template <int MODE>
__global__ void plan_kernel(CallArgs a)
{
    const int lane = threadIdx.x & 31;
    const uint32_t s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (s >= a.nseg) return;
    const gift_seg seg = a.segs[s];
    const uint32_t st = seg_prestatus<MODE>(a, seg, s, lane);
    if (lane == 0) {
        a.status[s] = st;
        a.acc[s] = make_uint4(0u, 0u, 0u, 0u);
        a.ticket[s] = 0u;
        a.wprefix[s] = st != 0 ? 0ull : seg_weight(seg_blocks(seg.len));      // the scan turns the weights into their prefix sum in place
        if (st != 0 && MODE == MODE_ENCRYPT) {
            reinterpret_cast<uint4*>(a.tags)[s] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
}

// ---------------------------------------------------------------------------
// 2. scan: the work split (split form)
// ---------------------------------------------------------------------------
//
// The cost of a block does not depend on the data, so the call is split statically: every
// accepted segment gets a weight, the weights are laid end to end, and resident warp w takes
// the weight range [w*slice, (w+1)*slice).  A segment's weight is its rows of 32 blocks plus
// SEG_WEIGHT for what a piece of work costs beyond its rows (pipeline fill, power fix-up, tag:
// about two rows, measured); its first SEG_WEIGHT units stand for that overhead, the rest
// map to its blocks.  A slice boundary inside a segment is rounded down to a whole row, so
// every warp's piece of a segment starts on a row.  Nothing is handed out at run time: no
// work counter, no imbalance from partial waves, and a warp touches as few segments as can be.

// One block.  A pass covers 8 192 segments: every warp takes 256 consecutive weights, lane l
// the elements l, l+32, ... of them, so that each load and store is one contiguous 256 bytes
// (with eight consecutive elements per thread a warp touches 16 lines per instruction and the
// load queue throttles: 60 us for 65 536 segments instead of about 10).
constexpr int SCAN_PER_THREAD = 8;

__global__ void scan_kernel(CallArgs a)
{
    __shared__ unsigned long long warp_sums[32];
    __shared__ unsigned long long carry;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    if (tid == 0) carry = 0ull;
    __syncthreads();
    const uint32_t per_pass = blockDim.x * SCAN_PER_THREAD;
    for (uint32_t base = 0; base < a.nseg; base += per_pass) {
        const uint32_t first = base + (uint32_t)wid * (32 * SCAN_PER_THREAD) + (uint32_t)lane;
        unsigned long long v[SCAN_PER_THREAD], inc[SCAN_PER_THREAD];
#pragma unroll
        for (int k = 0; k < SCAN_PER_THREAD; k++) {
            const uint32_t i = first + 32u * k;
            v[k] = i < a.nseg ? a.wprefix[i] : 0ull;          // the weight, written by the plan kernel
        }
        unsigned long long running = 0;                       // sum of the warp's rows before row k
#pragma unroll
        for (int k = 0; k < SCAN_PER_THREAD; k++) {
            unsigned long long x = v[k];
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, x, o);
                if (lane >= o) x += y;
            }
            inc[k] = running + x;                             // inclusive, inside the warp's 256
            running += __shfl_sync(0xFFFFFFFFu, x, 31);
        }
        if (lane == 0) warp_sums[wid] = running;
        __syncthreads();
        if (wid == 0) {
            unsigned long long w = lane < (int)(blockDim.x >> 5) ? warp_sums[lane] : 0ull;
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, w, o);
                if (lane >= o) w += y;
            }
            warp_sums[lane] = w;      // inclusive sums of the warps
        }
        __syncthreads();
        const unsigned long long off = carry + (wid ? warp_sums[wid - 1] : 0ull);
#pragma unroll
        for (int k = 0; k < SCAN_PER_THREAD; k++) {
            const uint32_t i = first + 32u * k;
            if (i < a.nseg) a.wprefix[i] = off + inc[k] - v[k];
        }
        __syncthreads();
        if (tid == 0) carry += warp_sums[(blockDim.x >> 5) - 1];
        __syncthreads();
    }
    if (tid == 0) {
        a.wprefix[a.nseg] = carry;
        unsigned long long slice = (carry + a.resident_warps - 1) / a.resident_warps;
        if (slice < MIN_SLICE) slice = MIN_SLICE;   // small calls: fewer warps rather than thinner slices
        a.glob->total_weight = carry;
        a.glob->slice = slice;
    }
}

// ---------------------------------------------------------------------------
// 3. crypt: the hot loop
// ---------------------------------------------------------------------------

extern __shared__ __align__(16) unsigned char smem_raw[];

// T-tables in shared memory, one copy per bank.  Entry x of table t for lane l is
// the word at byte  (t>>1)*65536 + x*256 + (t&1)*128 + l*4 : the index lands in
// byte 1 of the offset, so one byte-permute builds the address and the bank is
// always the lane's own.  With NT == 2 only T0 and T1 are stored; T2 and T3 are
// their 16-bit rotations.
template <int NT>
struct SmemTab {
    uint32_t lb0, lb1;     // lane*4 and lane*4 + 128
    // byte offset of entry (byte K of w) for this lane: index in byte 1, lane offset in byte 0
    template <int K>
    __device__ __forceinline__ uint32_t offset(uint32_t w, uint32_t lb) const
    {
        return __byte_perm(w, lb, 0x7604u | (K << 4));
    }
    template <int T, int K>
    __device__ __forceinline__ uint32_t look(uint32_t w) const
    {
        const uint32_t off = offset<K>(w, (T & 1) ? lb1 : lb0);
        if (NT == 4) {
            return *reinterpret_cast<const uint32_t*>(smem_raw + (T >> 1) * 65536 + off);
        } else {
            const uint32_t v = *reinterpret_cast<const uint32_t*>(smem_raw + off);
            return (T >> 1) ? __byte_perm(v, 0u, 0x1032u) : v;
        }
    }
    template <int K>
    __device__ __forceinline__ uint32_t sub(uint32_t w) const
    {
        return *reinterpret_cast<const uint32_t*>(smem_raw + offset<K>(w, lb0));
    }
};

// Word index inside a 64 KiB chunk: x*64 + parity*32 + lane.  A thread writes four
// consecutive lanes' copies of one entry with one 16-byte store; all its loads of the
// 1 KiB source table go out before the first store, so that their latency is paid once.
template <int NT>
__device__ __forceinline__ void fill_tables(const uint32_t* __restrict__ t0)
{
    uint4* tabs = reinterpret_cast<uint4*>(smem_raw);
    constexpr uint32_t quads = (NT == 4 ? 2u : 1u) * 4096u;
    constexpr int per_thread = (int)((quads + CRYPT_THREADS - 1) / CRYPT_THREADS);
    uint32_t v[per_thread];
#pragma unroll
    for (int k = 0; k < per_thread; k++) {
        const uint32_t idx = ((uint32_t)threadIdx.x + (uint32_t)k * CRYPT_THREADS) * 4u;
        v[k] = __ldg(t0 + ((idx >> 6) & 255u));
    }
#pragma unroll
    for (int k = 0; k < per_thread; k++) {
        const uint32_t q = (uint32_t)threadIdx.x + (uint32_t)k * CRYPT_THREADS;
        const uint32_t idx = q * 4u;
        const uint32_t chunk = idx >> 14, parity = (idx >> 5) & 1u;
        const uint32_t r = rotl32(v[k], 8 * (int)(chunk * 2 + parity));
        if (q < quads) tabs[q] = make_uint4(r, r, r, r);
    }
}

__device__ __forceinline__ uint32_t warp_xor(uint32_t v)
{
    for (int o = 16; o > 0; o >>= 1) v ^= __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

__device__ __forceinline__ void seg_nonce_words(const gift_seg& seg, uint32_t nonce[3])
{
    nonce[0] = (uint32_t)seg.nonce[0] | ((uint32_t)seg.nonce[1] << 8) | ((uint32_t)seg.nonce[2] << 16) | ((uint32_t)seg.nonce[3] << 24);
    nonce[1] = (uint32_t)seg.nonce[4] | ((uint32_t)seg.nonce[5] << 8) | ((uint32_t)seg.nonce[6] << 16) | ((uint32_t)seg.nonce[7] << 24);
    nonce[2] = (uint32_t)seg.nonce[8] | ((uint32_t)seg.nonce[9] << 8) | ((uint32_t)seg.nonce[10] << 16) | ((uint32_t)seg.nonce[11] << 24);
}

// Segments whose hash is complete wait here, per warp, until 32 of them can be finished at
// once.  Finishing a tag is one cipher block (E_K(J0)) and one field multiply (LEN * H) per
// segment; done right away it would occupy a whole warp for one segment's worth of work.  With
// one segment per lane the same instructions finish 32 tags, each lane reading its own
// segment's key material from global memory (the table lookups stay conflict-free: a lane
// always reads its own bank's copy).
struct Pending {
    uint4 sum[32];
    uint32_t seg[32];
};

// WRITE_OK: the status word of a segment whose tag is fine is written here (fused form: no
// plan kernel has written it before).
template <int MODE, bool WRITE_OK, class Tab>
__device__ __noinline__ void finish_pending(const CallArgs& a, const gift_seg* segtab, const Tab& tb, const Pending* pend,
                                            uint32_t n, int lane)
{
    bool ok = false;
    uint32_t s = 0;
    if ((uint32_t)lane < n) {
        s = pend->seg[lane];
        const uint4 sv = pend->sum[lane];
        const gift_seg seg = segtab[s];
        const KeyHot* hk = a.hot + seg.owner;
        u128 sum;
        sum.w[0] = sv.x; sum.w[1] = sv.y; sum.w[2] = sv.z; sum.w[3] = sv.w;
        uint32_t nonce[3];
        seg_nonce_words(seg, nonce);
        // the lane's round keys and hash subkey in one batch of loads (read one by one as the
        // rounds need them, their latency would sit on the tail of every call)
        uint32_t rkl[48];
#pragma unroll
        for (int q = 0; q < 12; q++) {
            const uint4 v = reinterpret_cast<const uint4*>(hk)[q];      // rk[0..43], then h[0..3]
            rkl[4 * q] = v.x; rkl[4 * q + 1] = v.y; rkl[4 * q + 2] = v.z; rkl[4 * q + 3] = v.w;
        }
        uint32_t tag[4];
        finish_tag(tb, rkl, rkl + 44, nonce, seg.len, sum, tag, a.aad ? a.aad + 16 * (size_t)s : nullptr,
                   a.pow + (size_t)seg.owner * (POW_LEVELS * 256));
        uint4* tagp = reinterpret_cast<uint4*>(a.tags) + s;
        if (MODE == MODE_ENCRYPT) {
            *tagp = make_uint4(tag[0], tag[1], tag[2], tag[3]);
            if (WRITE_OK) a.status[s] = 0u;
        } else {
            const uint4 given = *tagp;
            ok = given.x == tag[0] && given.y == tag[1] && given.z == tag[2] && given.w == tag[3];
            if (!ok) a.status[s] = GIFT_ST_TAG_MISMATCH;
            else if (WRITE_OK) a.status[s] = 0u;
        }
    }
    if (MODE == MODE_DECRYPT && a.owner_map != nullptr) {
        // import succeeded: record the claimed owner on the covered units, the warp taking
        // one verified segment at a time
        uint32_t m = __ballot_sync(0xFFFFFFFFu, ok);
        while (m) {
            const int k = __ffs(m) - 1;
            m &= m - 1;
            const uint32_t sk = __shfl_sync(0xFFFFFFFFu, s, k);
            const gift_seg seg = segtab[sk];
            uint64_t u0;
            const uint64_t nu = seg_unit_count(a, seg, &u0);
            for (uint64_t u = lane; u < nu; u += 32) a.owner_map[seg_unit(a, seg, u0, u)] = seg.owner;
        }
    }
}

// Fused form, per CTA: the descriptors of all segments, their weights and the exclusive prefix
// sum of the weights in shared memory (sseg[0..nseg), sp[0..nseg], sp[nseg] the total).  Only
// the descriptor checks that need no table walk decide a weight here; what else can refuse
// a segment (a bad page entry, the labels, a missing key, an overlap) is found by the warps
// whose slices touch it, which then skip it.  CTA 0 also writes the result of the segments
// refused here, which no slice touches.  Warp w takes the chunks of 32 segments w and
// w + 24; the loads are issued first (fused_load) so that their latency hides behind the
// table fill, the rest follows (fused_prefix).
constexpr int FUSED_CHUNKS_PER_WARP = (FUSED_MAX_SEGS / 32 + CRYPT_THREADS / 32 - 1) / (CRYPT_THREADS / 32);

__device__ __forceinline__ void fused_load(const CallArgs& a, gift_seg (&mine)[FUSED_CHUNKS_PER_WARP])
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int q = 0; q < FUSED_CHUNKS_PER_WARP; q++) {
        const uint32_t i = ((uint32_t)wid + (uint32_t)q * (CRYPT_THREADS / 32)) * 32u + (uint32_t)lane;
        if (i < a.nseg) mine[q] = a.segs[i];
    }
}

template <int MODE>
__device__ __forceinline__ void fused_prefix(const CallArgs& a, const gift_seg (&mine)[FUSED_CHUNKS_PER_WARP], gift_seg* sseg,
                                             unsigned long long* sp, unsigned long long* chunk_sums)
{
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    constexpr int NW = CRYPT_THREADS / 32;
    const uint32_t n_chunks = (a.nseg + 31u) >> 5;            // at most 32
#pragma unroll
    for (int q = 0; q < FUSED_CHUNKS_PER_WARP; q++) {
        const uint32_t c = (uint32_t)wid + (uint32_t)q * NW;
        if (c >= n_chunks) break;                             // uniform across the warp
        const uint32_t i = c * 32u + (uint32_t)lane;
        unsigned long long w = 0ull;
        if (i < a.nseg) {
            sseg[i] = mine[q];
            if (!desc_bad_quick(a, mine[q])) {
                w = seg_weight(seg_blocks(mine[q].len));
            } else if (blockIdx.x == 0) {
                a.status[i] = GIFT_ST_BAD_DESC;
                if (MODE == MODE_ENCRYPT) reinterpret_cast<uint4*>(a.tags)[i] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        unsigned long long x = w;
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, x, o);
            if (lane >= o) x += y;
        }
        if (i < a.nseg) sp[i] = x - w;                        // exclusive inside the chunk
        if (lane == 31) chunk_sums[c] = x;
    }
    __syncthreads();
    if (wid == 0) {
        unsigned long long w = (uint32_t)lane < n_chunks ? chunk_sums[lane] : 0ull;
        unsigned long long x = w;
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, x, o);
            if (lane >= o) x += y;
        }
        chunk_sums[lane] = x - w;                             // exclusive sums of the chunks
        if (lane == 31) sp[a.nseg] = x;                       // the total
    }
    __syncthreads();
    for (uint32_t i = tid; i < a.nseg; i += CRYPT_THREADS) sp[i] += chunk_sums[i >> 5];
    __syncthreads();
}

// PEEL: the first row of a piece runs without the (empty) hash update of a row before it.  Worth
// it where pieces are short; the second copy of the cipher code costs long pieces 2.6 %.
template <int MODE, int NT, bool FUSED, bool PEEL>
__global__ void __launch_bounds__(CRYPT_THREADS, 1) crypt_kernel(const __grid_constant__ CallArgs a, const uint32_t* __restrict__ t0)
{
    constexpr uint32_t TAB_BYTES = NT == 4 ? 131072u : 65536u;
    constexpr uint32_t NW = CRYPT_THREADS / 32;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    KeyHot* slot = reinterpret_cast<KeyHot*>(smem_raw + TAB_BYTES) + wid;
    Pending* pend = reinterpret_cast<Pending*>(smem_raw + TAB_BYTES + NW * sizeof(KeyHot)) + wid;
    unsigned long long* sp = reinterpret_cast<unsigned long long*>(smem_raw + TAB_BYTES + NW * (sizeof(KeyHot) + sizeof(Pending)));
    gift_seg* sseg = reinterpret_cast<gift_seg*>(sp + FUSED_MAX_SEGS + 1 + 32);
    const unsigned long long* prefix = FUSED ? sp : a.wprefix;
    const gift_seg* segtab = FUSED ? sseg : a.segs;

    // the call's total weight and the slice of a warp (see scan_kernel).  A CTA whose warps
    // all lie past the work leaves as soon as it knows.
    uint64_t total_weight, slice;
    if (FUSED) {
        gift_seg mine[FUSED_CHUNKS_PER_WARP];
        fused_load(a, mine);
        fill_tables<NT>(t0);                                 // no barrier needed before: disjoint shared memory
        fused_prefix<MODE>(a, mine, sseg, sp, sp + FUSED_MAX_SEGS + 1);      // ends with a barrier
        total_weight = sp[a.nseg];
        slice = (total_weight + a.resident_warps - 1) / a.resident_warps;
        if (slice < MIN_SLICE) slice = MIN_SLICE;
        if ((uint64_t)blockIdx.x * NW * slice >= total_weight) return;
    } else {
        total_weight = a.glob->total_weight;
        slice = a.glob->slice;
        if ((uint64_t)blockIdx.x * NW * slice >= total_weight) return;
        fill_tables<NT>(t0);
        __syncthreads();
    }
    SmemTab<NT> tb;
    tb.lb0 = (uint32_t)lane * 4u;
    tb.lb1 = (uint32_t)lane * 4u + 128u;
    uint32_t n_pend = 0;

    // this warp's share of the call: the weight range [g0, g1)
    const uint64_t g0 = (uint64_t)(blockIdx.x * NW + wid) * slice;
    if (g0 >= total_weight) return;
    const uint64_t g1 = g0 + slice < total_weight ? g0 + slice : total_weight;
    // first segment: the largest s with prefix[s] <= g0 (among equal prefixes the last one, which
    // is the one that has weight); the 32 lanes probe 32 points of the interval per step
    uint32_t s;
    {
        uint32_t lo = 0, hi = a.nseg;
        while (hi - lo > 1) {
            const uint32_t span = hi - lo - 1;                       // candidates lo+1 .. hi-1
            const uint32_t step = span / 32u + 1u;
            const uint32_t probe = lo + 1u + (uint32_t)lane * step;  // increasing with the lane
            const bool le = probe < hi && prefix[probe] <= g0;
            const uint32_t m = __ballot_sync(0xFFFFFFFFu, le);       // true on a prefix of the lanes
            const int k = __popc(m);
            const uint32_t next = lo + 1u + (uint32_t)k * step;      // first probe that said "greater"
            if (k) lo = lo + 1u + (uint32_t)(k - 1) * step;
            if (k < 32 && next < hi) hi = next;
        }
        s = lo;
    }
    for (; s < a.nseg; s++) {
        const uint64_t p0 = prefix[s];
        if (p0 >= g1) break;
        const uint64_t p1 = prefix[s + 1];
        if (p1 == p0) continue;                                      // refused before the split: no weight
        const gift_seg seg = segtab[s];
        if (FUSED) {
            // every warp that holds a piece of the segment reaches the same verdict on its own;
            // the one that holds the segment's first weight unit writes it down
            const uint32_t st = seg_prestatus<MODE>(a, seg, s, lane);
            if (st != 0) {
                if (g0 <= p0 && lane == 0) {
                    a.status[s] = st;
                    if (MODE == MODE_ENCRYPT) reinterpret_cast<uint4*>(a.tags)[s] = make_uint4(0u, 0u, 0u, 0u);
                }
                continue;
            }
        }
        const uint64_t nblk = seg_blocks(seg.len);
        // this warp's piece of the segment, and how many warps have one (each reports once,
        // with or without blocks; the last report finishes the tag)
        const SlicePiece piece = slice_piece(g0, g1, p0, p1, nblk, slice);
        const uint64_t run_first = piece.first;
        const uint32_t run_n = (uint32_t)(piece.end - piece.first);
        const uint32_t seg_runs = piece.reporters;

        // this warp's copy of the owner's key material (512 bytes: one uint4 per lane)
        __syncwarp();
        reinterpret_cast<uint4*>(slot)[lane] = reinterpret_cast<const uint4*>(a.hot + seg.owner)[lane];
        __syncwarp();
        const uint32_t* rk = slot->rk;
        uint32_t nonce[3];
        seg_nonce_words(seg, nonce);
        const CtrPrefix pre = ctr_prefix(tb, rk, nonce);
        SegAddr addr;
        addr.table = a.page_table;
        addr.page_bytes = a.page_bytes;
        addr.origin = a.page_table ? (uint64_t)seg.page0 : seg.offset;

        u128 part = gf_zero();
        if (run_n == 0) {
            // a piece without blocks (an empty segment, or a slice boundary inside the segment's
            // overhead weight or its last partial row): nothing to read, only the report below
        } else if (a.page_table == nullptr || (a.page_bytes & 511) == 0) {
            // rows of 32 blocks never straddle a page: the pipelined row loop applies
            part = run_lane_rows<MODE, PEEL>(tb, rk, pre, slot->hs, a.pow + (size_t)seg.owner * (POW_LEVELS * 256),
                                       a.src, a.dst, addr, nblk, run_first, run_n, (uint32_t)(seg.len & 15), lane);
        } else {
            part = run_lane<1, MODE>(tb, rk, pre, slot->hs, a.pow + (size_t)seg.owner * (POW_LEVELS * 256),
                                     a.src, a.dst, addr, nblk, run_first, run_n, (uint32_t)(seg.len & 15), lane);
        }
        u128 sum;
        sum.w[0] = warp_xor(part.w[0]);
        sum.w[1] = warp_xor(part.w[1]);
        sum.w[2] = warp_xor(part.w[2]);
        sum.w[3] = warp_xor(part.w[3]);

        // combine the pieces of a segment: XOR is order-free, the last arrival finishes and
        // leaves the accumulator and the ticket at zero for the next call
        bool last = true;
        if (seg_runs > 1) {
            uint32_t t = 0;
            if (lane == 0) {
                uint32_t* acc = reinterpret_cast<uint32_t*>(a.acc + s);
                atomicXor(acc + 0, sum.w[0]);
                atomicXor(acc + 1, sum.w[1]);
                atomicXor(acc + 2, sum.w[2]);
                atomicXor(acc + 3, sum.w[3]);
                __threadfence();
                t = atomicAdd(a.ticket + s, 1u);
            }
            t = __shfl_sync(0xFFFFFFFFu, t, 0);
            last = t == seg_runs - 1;
            if (last) {
                __threadfence();
                uint32_t* acc = reinterpret_cast<uint32_t*>(a.acc + s);
                if (lane < 4) sum.w[0] = atomicExch(acc + lane, 0u);
                if (lane == 4) a.ticket[s] = 0u;
                const uint32_t v = sum.w[0];
                sum.w[0] = __shfl_sync(0xFFFFFFFFu, v, 0);
                sum.w[1] = __shfl_sync(0xFFFFFFFFu, v, 1);
                sum.w[2] = __shfl_sync(0xFFFFFFFFu, v, 2);
                sum.w[3] = __shfl_sync(0xFFFFFFFFu, v, 3);
            }
        }
        if (last) {
            if (lane == 0) {
                pend->sum[n_pend] = make_uint4(sum.w[0], sum.w[1], sum.w[2], sum.w[3]);
                pend->seg[n_pend] = s;
            }
            n_pend++;
            if (n_pend == 32u) {
                __syncwarp();
                finish_pending<MODE, FUSED>(a, segtab, tb, pend, n_pend, lane);
                __syncwarp();
                n_pend = 0;
            }
        }
    }
    __syncwarp();
    if (n_pend) finish_pending<MODE, FUSED>(a, segtab, tb, pend, n_pend, lane);
}

// Shared memory of one CTA of the cipher kernel.
template <int NT, bool FUSED>
constexpr size_t crypt_smem_bytes()
{
    return (NT == 4 ? 131072u : 65536u) + (CRYPT_THREADS / 32) * (sizeof(KeyHot) + sizeof(Pending)) +
           (FUSED ? (FUSED_MAX_SEGS + 1 + 32) * sizeof(unsigned long long) + FUSED_MAX_SEGS * sizeof(gift_seg) : 0);
}

// ---------------------------------------------------------------------------
// 4. fix-up after decrypt: failed segments read as zeros and become unowned
// ---------------------------------------------------------------------------

__global__ void fixup_kernel(CallArgs a)
{
    for (uint32_t s = blockIdx.x; s < a.nseg; s += gridDim.x) {
        const uint32_t st = a.status[s];
        if ((st & (GIFT_ST_TAG_MISMATCH | GIFT_ST_NO_KEY)) == 0 || (st & (GIFT_ST_BAD_DESC | GIFT_ST_OVERLAP))) continue;
        const gift_seg seg = a.segs[s];
        const uint64_t full = seg.len >> 4;
        if (a.page_table == nullptr) {
            uint4* p = reinterpret_cast<uint4*>(a.dst + seg.offset);
            for (uint64_t k = threadIdx.x; k < full; k += blockDim.x) p[k] = make_uint4(0u, 0u, 0u, 0u);
            for (uint64_t k = (full << 4) + threadIdx.x; k < seg.len; k += blockDim.x) a.dst[seg.offset + k] = 0;
        } else {
            const uint64_t per_page = a.page_bytes >> 4;
            for (uint64_t k = threadIdx.x; k < full; k += blockDim.x) {
                const uint64_t pg = k / per_page, in = k - pg * per_page;
                const uint64_t base = (uint64_t)(uint32_t)a.page_table[(uint64_t)seg.page0 + pg] * a.page_bytes;
                reinterpret_cast<uint4*>(a.dst + base)[in] = make_uint4(0u, 0u, 0u, 0u);
            }
            for (uint64_t k = (full << 4) + threadIdx.x; k < seg.len; k += blockDim.x) {
                const uint64_t pg = k / a.page_bytes, in = k - pg * a.page_bytes;
                const uint64_t base = (uint64_t)(uint32_t)a.page_table[(uint64_t)seg.page0 + pg] * a.page_bytes;
                a.dst[base + in] = 0;
            }
        }
        if (a.owner_map != nullptr) {
            uint64_t u0;
            const uint64_t nu = seg_unit_count(a, seg, &u0);
            for (uint64_t k = threadIdx.x; k < nu; k += blockDim.x)
                a.owner_map[seg_unit(a, seg, u0, k)] = GIFT_OWNER_NONE;
        }
    }
}

}  // namespace gift

// ---------------------------------------------------------------------------
// optional overlap check of a segment table (paper sec. 4.3 rule step 3: tensors occupy
// distinct memory unless meant to alias; sec. 3 step 4: every byte has one owner)
// ---------------------------------------------------------------------------
//
// Off unless the ctx was created with GIFT_CTX_CHECK_OVERLAP.  A segment that shares a byte
// with another valid segment of the call, or that lists one physical page twice, is flagged
// in overlap[]; the plan then refuses it with GIFT_ST_OVERLAP.  Segments with a bad
// descriptor and empty segments take no part.  Nothing waits on anything.
namespace gift {

// Flat mode: all pairs.  One thread per segment i; the table passes through shared memory
// in tiles.  65 536 segments are 4.3 G interval tests, a fraction of a millisecond.
constexpr int OVL_TILE = 256;

__global__ void __launch_bounds__(OVL_TILE) overlap_flat_kernel(CallArgs a, uint8_t* overlap)
{
    __shared__ unsigned long long lo_s[OVL_TILE], hi_s[OVL_TILE];
    const uint32_t i = blockIdx.x * OVL_TILE + threadIdx.x;
    unsigned long long lo = 1, hi = 0;                       // lo >= hi: takes no part
    if (i < a.nseg) {
        const gift_seg seg = a.segs[i];
        if (!desc_bad_quick(a, seg) && seg.len > 0) { lo = seg.offset; hi = seg.offset + seg.len; }
    }
    bool hit = false;
    for (uint32_t base = 0; base < a.nseg; base += OVL_TILE) {
        const uint32_t j = base + threadIdx.x;
        unsigned long long l = 1, h = 0;
        if (j < a.nseg) {
            const gift_seg seg = a.segs[j];
            if (!desc_bad_quick(a, seg) && seg.len > 0) { l = seg.offset; h = seg.offset + seg.len; }
        }
        __syncthreads();
        lo_s[threadIdx.x] = l;
        hi_s[threadIdx.x] = h;
        __syncthreads();
        if (lo < hi) {
#pragma unroll 8
            for (int k = 0; k < OVL_TILE; k++) {
                const bool other = base + (uint32_t)k != i;
                hit |= other && lo_s[k] < hi && lo < hi_s[k] && lo_s[k] < hi_s[k];
            }
        }
    }
    if (i < a.nseg) overlap[i] = hit ? 1 : 0;
}

// Paged mode: two segments share bytes exactly when they share a physical page (every page
// of a chain is used from its first byte).  One warp per segment claims its pages in
// claim[] (all -1 before the launch); whoever finds a page taken flags itself and the
// first claimant.  overlap[] is zero before the launch.
__global__ void overlap_paged_kernel(CallArgs a, int32_t* claim, uint8_t* overlap)
{
    const int lane = threadIdx.x & 31;
    const uint32_t s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (s >= a.nseg) return;
    const gift_seg seg = a.segs[s];
    if (desc_bad_quick(a, seg)) return;
    const bool labels = a.owner_map != nullptr;
    const uint64_t np = (seg.len + a.page_bytes - 1) / a.page_bytes;
    bool b = false;
    for (uint64_t k = lane; k < np; k += 32) {
        const int32_t t = a.page_table[(uint64_t)seg.page0 + k];
        b |= t < 0 || ((uint64_t)t + 1) * a.page_bytes > a.buf_bytes || (labels && (uint64_t)t >= a.n_units);
    }
    if (__any_sync(0xFFFFFFFFu, b)) return;                  // a bad descriptor claims nothing
    for (uint64_t k = lane; k < np; k += 32) {
        const int32_t t = a.page_table[(uint64_t)seg.page0 + k];
        const int32_t old = atomicCAS(claim + t, -1, (int32_t)s);
        if (old != -1) {
            overlap[s] = 1;
            if ((uint32_t)old != s) overlap[old] = 1;
        }
    }
}

}  // namespace gift
