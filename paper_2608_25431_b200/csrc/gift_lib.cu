// libgift: context, kernels and C entry points (see include/gift.h).
//
// Call structure of gift_seg_encrypt / gift_seg_decrypt / gift_verify_tags, all
// on the caller's stream with no host round trip in between:
//   1. plan_kernel     one warp per segment: descriptor checks, ownership-label
//                      check, pre-status, zeroed hash accumulators
//   2. scan_kernel     prefix sum of the accepted segments' weights and the weight
//                      slice of a resident warp (the static work split)
//   3. crypt_kernel    every resident warp takes its slice; per piece of a segment:
//                      CTR keystream + XOR + GHASH; the warp whose report completes
//                      a segment finishes its tag (no waiting, tickets only)
//   4. fixup_kernel    decrypt only: zero-fills failed segments, marks their units
//
// AES uses T-tables replicated across the 32 shared-memory banks so that a warp's
// 32 data-dependent lookups never conflict; GHASH uses masked integer multiplies
// (gf128.cuh).  The path is bound by the integer pipes, not by HBM: about one eighth
// of the memory bandwidth is needed, so data moves with plain 128-bit
// loads and stores and no staging through shared memory.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "../../include/gift.h"
#include "gift_core.cuh"

using namespace gift;

#define GIFT_VERSION 100u   // 0.1.0

#include "gift_internal.cuh"
#include "gift_rules.cuh"

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
    unsigned long long* wprefix;   // [nseg + 1] exclusive prefix of the segment weights
    uint4* acc;
    uint32_t* ticket;
    Globals* glob;
    uint32_t resident_warps;       // warps of the cipher kernel on the whole GPU
};

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
// 1. plan: validation, label check (paper sec. 3 step 4, sec. 4.2), pre-status
// ---------------------------------------------------------------------------

template <int MODE>
__global__ void plan_kernel(CallArgs a)
{
    const int lane = threadIdx.x & 31;
    const uint32_t s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (s >= a.nseg) return;
    const gift_seg seg = a.segs[s];
    const bool labels = a.owner_map != nullptr;

    bool bad = seg.flags != 0 || seg.len > GIFT_MAX_SEG_BYTES;
    if (!bad) {
        if (a.page_table == nullptr) {
            bad = (seg.offset & 15) != 0 || seg.offset > a.buf_bytes || seg.len > a.buf_bytes - seg.offset;
            if (!bad && labels && seg.len > 0) {
                const uint64_t u1 = (seg.offset + seg.len + a.unit_bytes - 1) / a.unit_bytes;
                bad = u1 > a.n_units;
            }
        } else {
            const uint64_t np = (seg.len + a.page_bytes - 1) / a.page_bytes;
            bad = (uint64_t)seg.page0 + np > a.n_pages;
            if (!bad) {
                bool b = false;
                for (uint64_t k = lane; k < np; k += 32) {
                    const int32_t t = a.page_table[(uint64_t)seg.page0 + k];
                    b |= t < 0 || ((uint64_t)t + 1) * a.page_bytes > a.buf_bytes ||
                         (labels && (uint64_t)t >= a.n_units);
                }
                bad = __any_sync(0xFFFFFFFFu, b);
            }
        }
    }
    uint32_t st = 0;
    if (bad) {
        st = GIFT_ST_BAD_DESC;
    } else {
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
    }
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
// 2. scan: the work split
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
#ifndef GIFT_K3_ON_MUL
#define GIFT_K3_ON_MUL 0   // measured: the two extra issue slots cost more than the freed logic slot (406 vs 421 GB/s)
#endif

template <int NT>
struct SmemTab {
    uint32_t lb0, lb1;     // lane*4 and lane*4 + 128
    // byte offset of entry (byte K of w) for this lane: index in byte 1, lane offset in byte 0
    template <int K>
    __device__ __forceinline__ uint32_t offset(uint32_t w, uint32_t lb) const
    {
#if GIFT_K3_ON_MUL
        if (K == 3) {
            // the top byte through the multiply pipe: (w * 256) >> 32 = w >> 24, then * 256 + lane offset
            const uint32_t k256 = GIFT_KMUL(4);
            const uint32_t top = (uint32_t)(((uint64_t)w * k256) >> 32);
            return top * k256 + lb;
        }
#endif
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

template <int NT>
__device__ __forceinline__ void fill_tables(const uint32_t* __restrict__ t0)
{
    // word index inside a 64 KiB chunk: x*64 + parity*32 + lane
    uint32_t* tabs = reinterpret_cast<uint32_t*>(smem_raw);
    constexpr int chunks = NT == 4 ? 2 : 1;
    for (uint32_t idx = threadIdx.x; idx < chunks * 16384u; idx += blockDim.x) {
        const uint32_t chunk = idx >> 14, x = (idx >> 6) & 255u, parity = (idx >> 5) & 1u;
        const uint32_t t = chunk * 2 + parity;
        tabs[idx] = rotl32(t0[x], 8 * (int)t);
    }
}

__device__ __forceinline__ uint32_t warp_xor(uint32_t v)
{
    for (int o = 16; o > 0; o >>= 1) v ^= __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
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

template <int MODE, class Tab>
__device__ __noinline__ void finish_pending(const CallArgs& a, const Tab& tb, const Pending* pend, uint32_t n, int lane)
{
    bool ok = false;
    uint32_t s = 0;
    if ((uint32_t)lane < n) {
        s = pend->seg[lane];
        const uint4 sv = pend->sum[lane];
        const gift_seg seg = a.segs[s];
        const KeyHot* hk = a.hot + seg.owner;
        u128 sum;
        sum.w[0] = sv.x; sum.w[1] = sv.y; sum.w[2] = sv.z; sum.w[3] = sv.w;
        uint32_t nonce[3];
        nonce[0] = (uint32_t)seg.nonce[0] | ((uint32_t)seg.nonce[1] << 8) | ((uint32_t)seg.nonce[2] << 16) | ((uint32_t)seg.nonce[3] << 24);
        nonce[1] = (uint32_t)seg.nonce[4] | ((uint32_t)seg.nonce[5] << 8) | ((uint32_t)seg.nonce[6] << 16) | ((uint32_t)seg.nonce[7] << 24);
        nonce[2] = (uint32_t)seg.nonce[8] | ((uint32_t)seg.nonce[9] << 8) | ((uint32_t)seg.nonce[10] << 16) | ((uint32_t)seg.nonce[11] << 24);
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
        } else {
            const uint4 given = *tagp;
            ok = given.x == tag[0] && given.y == tag[1] && given.z == tag[2] && given.w == tag[3];
            if (!ok) a.status[s] = GIFT_ST_TAG_MISMATCH;
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
            const gift_seg seg = a.segs[sk];
            uint64_t u0;
            const uint64_t nu = seg_unit_count(a, seg, &u0);
            for (uint64_t u = lane; u < nu; u += 32) a.owner_map[seg_unit(a, seg, u0, u)] = seg.owner;
        }
    }
}

template <int U, int MODE, int NT, int THREADS>
__global__ void __launch_bounds__(THREADS, 1) crypt_kernel(const __grid_constant__ CallArgs a, const uint32_t* __restrict__ t0)
{
    constexpr uint32_t TAB_BYTES = NT == 4 ? 131072u : 65536u;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    fill_tables<NT>(t0);
    __syncthreads();
    SmemTab<NT> tb;
    tb.lb0 = (uint32_t)lane * 4u;
    tb.lb1 = (uint32_t)lane * 4u + 128u;
    KeyHot* slot = reinterpret_cast<KeyHot*>(smem_raw + TAB_BYTES) + wid;
    Pending* pend = reinterpret_cast<Pending*>(smem_raw + TAB_BYTES + (THREADS / 32) * sizeof(KeyHot)) + wid;
    uint32_t n_pend = 0;

    // this warp's share of the call: the weight range [g0, g1) (see scan_kernel)
    const uint64_t total_weight = a.glob->total_weight, slice = a.glob->slice;
    const uint64_t g0 = (uint64_t)(blockIdx.x * (THREADS / 32) + wid) * slice;
    if (g0 >= total_weight) return;
    const uint64_t g1 = g0 + slice < total_weight ? g0 + slice : total_weight;
    // first segment: the largest s with wprefix[s] <= g0 (among equal prefixes the last one, which
    // is the one that has weight); the 32 lanes probe 32 points of the interval per step
    uint32_t s;
    {
        uint32_t lo = 0, hi = a.nseg;
        while (hi - lo > 1) {
            const uint32_t span = hi - lo - 1;                       // candidates lo+1 .. hi-1
            const uint32_t step = span / 32u + 1u;
            const uint32_t probe = lo + 1u + (uint32_t)lane * step;  // increasing with the lane
            const bool le = probe < hi && a.wprefix[probe] <= g0;
            const uint32_t m = __ballot_sync(0xFFFFFFFFu, le);       // true on a prefix of the lanes
            const int k = __popc(m);
            const uint32_t next = lo + 1u + (uint32_t)k * step;      // first probe that said "greater"
            if (k) lo = lo + 1u + (uint32_t)(k - 1) * step;
            if (k < 32 && next < hi) hi = next;
        }
        s = lo;
    }
    for (; s < a.nseg; s++) {
        const uint64_t p0 = a.wprefix[s];
        if (p0 >= g1) break;
        const uint64_t p1 = a.wprefix[s + 1];
        if (p1 == p0) continue;                                      // rejected by the plan: no weight
        const gift_seg seg = a.segs[s];
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
        nonce[0] = (uint32_t)seg.nonce[0] | ((uint32_t)seg.nonce[1] << 8) | ((uint32_t)seg.nonce[2] << 16) | ((uint32_t)seg.nonce[3] << 24);
        nonce[1] = (uint32_t)seg.nonce[4] | ((uint32_t)seg.nonce[5] << 8) | ((uint32_t)seg.nonce[6] << 16) | ((uint32_t)seg.nonce[7] << 24);
        nonce[2] = (uint32_t)seg.nonce[8] | ((uint32_t)seg.nonce[9] << 8) | ((uint32_t)seg.nonce[10] << 16) | ((uint32_t)seg.nonce[11] << 24);
        const CtrPrefix pre = ctr_prefix(tb, rk, nonce);
        SegAddr addr;
        addr.table = a.page_table;
        addr.page_bytes = a.page_bytes;
        addr.origin = a.page_table ? (uint64_t)seg.page0 : seg.offset;

        u128 part = gf_zero();
        if (run_n == 0) {
            // a piece without blocks (an empty segment, or a slice boundary inside the segment's
            // overhead weight or its last partial row): nothing to read, only the report below
        } else if (U == 1 && (a.page_table == nullptr || (a.page_bytes & 511) == 0)) {
            // rows of 32 blocks never straddle a page: the pipelined row loop applies
            part = run_lane_rows<MODE>(tb, rk, pre, slot->hs[0], a.pow + (size_t)seg.owner * (POW_LEVELS * 256),
                                       a.src, a.dst, addr, nblk, run_first, run_n, (uint32_t)(seg.len & 15), lane);
        } else {
            part = run_lane<U, MODE>(tb, rk, pre, slot->hs[U - 1], a.pow + (size_t)seg.owner * (POW_LEVELS * 256),
                                     a.src, a.dst, addr, nblk, run_first, run_n, (uint32_t)(seg.len & 15), lane);
        }
        u128 sum;
        sum.w[0] = warp_xor(part.w[0]);
        sum.w[1] = warp_xor(part.w[1]);
        sum.w[2] = warp_xor(part.w[2]);
        sum.w[3] = warp_xor(part.w[3]);

        // combine the runs of a segment: XOR is order-free, the last arrival finishes
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
                if (lane < 4) sum.w[0] = atomicOr(acc + lane, 0u);
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
                finish_pending<MODE>(a, tb, pend, n_pend, lane);
                __syncwarp();
                n_pend = 0;
            }
        }
    }
    __syncwarp();
    if (n_pend) finish_pending<MODE>(a, tb, pend, n_pend, lane);
}

// ---------------------------------------------------------------------------
// 4. fix-up after decrypt: failed segments read as zeros and become unowned
// ---------------------------------------------------------------------------

__global__ void fixup_kernel(CallArgs a)
{
    for (uint32_t s = blockIdx.x; s < a.nseg; s += gridDim.x) {
        const uint32_t st = a.status[s];
        if ((st & (GIFT_ST_TAG_MISMATCH | GIFT_ST_NO_KEY)) == 0 || (st & GIFT_ST_BAD_DESC)) continue;
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

// ---------------------------------------------------------------------------
// label propagation (paper sec. 4.3, rule steps 4 and 5)
// ---------------------------------------------------------------------------

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

// One warp per reduction segment; outputs outside every segment become CONFLICT.
__global__ void rule_segreduce_kernel(RuleArgs r)
{
    const int lane = threadIdx.x & 31;
    const uint32_t w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
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
        const uint32_t extra = (blockIdx.x * blockDim.x + threadIdx.x) - r.n_seg * 32u;
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

__global__ void viol_init_kernel(uint32_t* viol)
{
    viol[0] = 0u;
    viol[1] = 0xFFFFFFFFu;
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------

int ensure_scratch(gift_ctx* c, uint32_t nseg)
{
    if (nseg <= c->seg_cap) return GIFT_OK;
    uint32_t cap = c->seg_cap ? c->seg_cap : 1024u;
    while (cap < nseg) cap = cap > 0x7FFFFFFFu ? nseg : cap * 2u;
    CU_TRY(cudaDeviceSynchronize());
    cudaFree(c->d_wprefix);
    cudaFree(c->d_acc);
    cudaFree(c->d_ticket);
    c->d_wprefix = nullptr; c->d_acc = nullptr; c->d_ticket = nullptr;
    c->seg_cap = 0;
    CU_TRY(cudaMalloc(&c->d_wprefix, ((size_t)cap + 1) * sizeof(unsigned long long)));
    CU_TRY(cudaMalloc(&c->d_acc, (size_t)cap * sizeof(uint4)));
    CU_TRY(cudaMalloc(&c->d_ticket, (size_t)cap * sizeof(uint32_t)));
    c->seg_cap = cap;
    return GIFT_OK;
}

template <int U, int MODE, int NT, int THREADS>
int launch_crypt_t(gift_ctx* c, const CallArgs& a, cudaStream_t st)
{
    const size_t smem = (NT == 4 ? 131072u : 65536u) + (THREADS / 32) * (sizeof(KeyHot) + sizeof(Pending));
    static bool configured[8] = {false, false, false, false, false, false, false, false};
    auto kern = crypt_kernel<U, MODE, NT, THREADS>;
    if (c->device < 8 && !configured[c->device]) {
        CU_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured[c->device] = true;
    } else if (c->device >= 8) {
        CU_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    }
    const bool timed = c->timing && c->ev && c->n_timed < MAX_TIMED;
    if (timed) CU_TRY(cudaEventRecord(c->ev[2 * c->n_timed], st));
    kern<<<c->num_sms, THREADS, smem, st>>>(a, c->d_t0);
    if (timed) {
        CU_TRY(cudaEventRecord(c->ev[2 * c->n_timed + 1], st));
        c->n_timed++;
    }
    c->launches++;
    return GIFT_OK;
}

template <int MODE>
int launch_crypt(gift_ctx* c, const CallArgs& a, cudaStream_t st)
{
    if (c->threads == 1024) {
        if (c->tables == 4) return launch_crypt_t<1, MODE, 4, 1024>(c, a, st);
        return launch_crypt_t<1, MODE, 2, 1024>(c, a, st);
    }
    if (c->threads == 768) {
        if (c->tables == 4) return launch_crypt_t<1, MODE, 4, 768>(c, a, st);
        return launch_crypt_t<1, MODE, 2, 768>(c, a, st);
    }
    if (c->tables == 4) {
        return c->chains == 2 ? launch_crypt_t<2, MODE, 4, 512>(c, a, st) : launch_crypt_t<1, MODE, 4, 512>(c, a, st);
    }
    return c->chains == 2 ? launch_crypt_t<2, MODE, 2, 512>(c, a, st) : launch_crypt_t<1, MODE, 2, 512>(c, a, st);
}

template <int MODE>
int seg_call(gift_ctx* c, const void* src, void* dst, uint64_t buf_bytes, const gift_seg* segs, uint32_t nseg,
             const gift_pages* pages, const gift_labels* labels, uint8_t* tags, uint32_t* status, void* stream)
{
    if (!c || !segs || !tags || !status) return nseg == 0 && c ? GIFT_OK : GIFT_E_INVAL;
    if (nseg == 0) return GIFT_OK;
    if (!src || (MODE != MODE_VERIFY && !dst)) return GIFT_E_INVAL;
    if (((uintptr_t)src & 15) || ((uintptr_t)dst & 15) || ((uintptr_t)tags & 15)) return GIFT_E_ALIGN;
    if (pages && (!pages->table || pages->page_bytes == 0)) return GIFT_E_INVAL;
    if (pages && (pages->page_bytes & 15)) return GIFT_E_ALIGN;
    if (labels && (!labels->owner_map || (!pages && labels->unit_bytes == 0))) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    int rc = ensure_scratch(c, nseg);
    if (rc != GIFT_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;

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
    a.aad = c->aad;
    a.status = status;
    a.hot = c->d_hot;
    a.pow = c->d_pow;
    a.max_users = c->max_users;
    a.wprefix = c->d_wprefix;
    a.acc = c->d_acc;
    a.ticket = c->d_ticket;
    a.glob = c->d_glob;
    a.resident_warps = (uint32_t)c->num_sms * (uint32_t)(c->threads / 32);

    CU_TRY(cudaMemsetAsync(c->d_glob, 0, sizeof(Globals), st));
    const uint32_t plan_blocks = (nseg + 7) / 8;          // 8 warps per block, one warp per segment
    plan_kernel<MODE><<<plan_blocks, 256, 0, st>>>(a);
    scan_kernel<<<1, 1024, 0, st>>>(a);
    c->launches += 2;
    rc = launch_crypt<MODE>(c, a, st);
    if (rc != GIFT_OK) return rc;
    if (MODE == MODE_DECRYPT) {
        uint32_t fb = nseg < (uint32_t)c->num_sms * 8u ? nseg : (uint32_t)c->num_sms * 8u;
        fixup_kernel<<<fb, 256, 0, st>>>(a);
        c->launches++;
    }
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}

}  // namespace

// ---------------------------------------------------------------------------
// C entry points
// ---------------------------------------------------------------------------

extern "C" {

int gift_ctx_create(gift_ctx** out, int device, uint32_t max_users, uint32_t flags)
{
    if (!out || max_users == 0) return GIFT_E_INVAL;
    *out = nullptr;
    int chains = (int)(flags & 0xFu), tables = (int)((flags >> 4) & 0xFu), threads = (int)((flags >> 8) & 0xFu) * 256;
    if (chains == 0) chains = 1;
    if (tables == 0) tables = 4;
    if (threads == 0) threads = chains == 2 ? 512 : 768;
    if ((chains != 1 && chains != 2) || (tables != 2 && tables != 4) || (threads != 512 && threads != 768 && threads != 1024) ||
        (threads > 512 && chains != 1) || (flags >> 12))
        return GIFT_E_INVAL;
    if (max_users > (1u << 20)) return GIFT_E_RANGE;
    DeviceGuard g(device);
    if (!g.ok) return GIFT_E_CUDA;
    gift_ctx* c = new (std::nothrow) gift_ctx();
    if (!c) return GIFT_E_NOMEM;
    memset(c, 0, sizeof(*c));
    c->device = device;
    c->max_users = max_users;
    c->flags = flags;
    c->chains = chains;
    c->tables = tables;
    c->threads = threads;
    int rc = GIFT_OK;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete c; return GIFT_E_CUDA; }
    c->num_sms = prop.multiProcessorCount;
    auto fail = [&](int code) { gift_ctx_destroy(c); return code; };
    if (cudaMalloc(&c->d_t0, 256 * sizeof(uint32_t)) != cudaSuccess) return fail(GIFT_E_NOMEM);
    if (cudaMalloc(&c->d_isbox, 256) != cudaSuccess) return fail(GIFT_E_NOMEM);
    if (cudaMalloc(&c->d_hot, (size_t)max_users * sizeof(KeyHot)) != cudaSuccess) return fail(GIFT_E_NOMEM);
    if (cudaMalloc(&c->d_pow, (size_t)max_users * POW_LEVELS * 256 * sizeof(u128)) != cudaSuccess) return fail(GIFT_E_NOMEM);
    if (cudaMalloc(&c->d_glob, sizeof(Globals)) != cudaSuccess) return fail(GIFT_E_NOMEM);
    if (cudaMemset(c->d_hot, 0, (size_t)max_users * sizeof(KeyHot)) != cudaSuccess) return fail(GIFT_E_CUDA);
    if (cudaMemset(c->d_pow, 0, (size_t)max_users * POW_LEVELS * 256 * sizeof(u128)) != cudaSuccess) return fail(GIFT_E_CUDA);
    if (cudaMemset(c->d_glob, 0, sizeof(Globals)) != cudaSuccess) return fail(GIFT_E_CUDA);
    init_t0_kernel<<<1, 256>>>(c->d_t0, c->d_isbox);
    c->launches++;
    if (cudaDeviceSynchronize() != cudaSuccess) return fail(GIFT_E_CUDA);
    rc = ensure_scratch(c, 1024);
    if (rc != GIFT_OK) return fail(rc);
    *out = c;
    return GIFT_OK;
}

int gift_ctx_destroy(gift_ctx* c)
{
    if (!c) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (g.ok) {
        cudaDeviceSynchronize();
        if (c->d_hot) cudaMemset(c->d_hot, 0, (size_t)c->max_users * sizeof(KeyHot));
        if (c->d_pow) cudaMemset(c->d_pow, 0, (size_t)c->max_users * POW_LEVELS * 256 * sizeof(u128));
        if (c->d_stage_keys) cudaMemset(c->d_stage_keys, 0, (size_t)c->stage_cap * 16);
        cudaDeviceSynchronize();
        cudaFree(c->d_t0); cudaFree(c->d_isbox); cudaFree(c->d_hot); cudaFree(c->d_pow); cudaFree(c->d_glob);
        cudaFree(c->d_wprefix); cudaFree(c->d_acc); cudaFree(c->d_ticket);
        cudaFree(c->d_stage_ids); cudaFree(c->d_stage_keys); cudaFree(c->d_snapshot); cudaFree(c->d_next_sync);
        if (c->h_stage) {
            memset(c->h_stage, 0, (size_t)c->stage_cap * 20);
            cudaFreeHost(c->h_stage);
        }
        if (c->ev) {
            for (uint32_t i = 0; i < 2 * MAX_TIMED; i++) cudaEventDestroy(c->ev[i]);
            delete[] c->ev;
        }
    }
    delete c;
    return GIFT_OK;
}

int gift_ctx_reserve(gift_ctx* c, uint32_t max_segs)
{
    if (!c) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    return ensure_scratch(c, max_segs);
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
    return seg_call<MODE_ENCRYPT>(c, src, dst, buf_bytes, segs, nseg, pages, labels, tags_out, status, stream);
}

int gift_seg_decrypt(gift_ctx* c, const void* src, void* dst, uint64_t buf_bytes, const gift_seg* segs,
                     uint32_t nseg, const gift_pages* pages, gift_labels* labels, const uint8_t* tags_in,
                     uint32_t* status, void* stream)
{
    return seg_call<MODE_DECRYPT>(c, src, dst, buf_bytes, segs, nseg, pages, labels, (uint8_t*)tags_in, status, stream);
}

int gift_verify_tags(gift_ctx* c, const void* src, uint64_t buf_bytes, const gift_seg* segs, uint32_t nseg,
                     const gift_pages* pages, const uint8_t* tags_in, uint32_t* status, void* stream)
{
    return seg_call<MODE_VERIFY>(c, src, nullptr, buf_bytes, segs, nseg, pages, nullptr, (uint8_t*)tags_in, status, stream);
}

int gift_propagate_labels(gift_ctx* c, const gift_rule* rule, const int32_t* const* in_maps, int32_t* out,
                          uint32_t* viol, void* stream)
{
    if (!c) return GIFT_E_INVAL;
    RuleArgs r;
    const int rc = fill_rule_args(rule, in_maps, out, viol, r);
    if (rc != GIFT_OK) return rc;
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
    viol_init_kernel<<<1, 1, 0, st>>>(viol);
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

int gift_ctx_bind_aad(gift_ctx* c, const uint8_t* aad16)
{
    if (!c) return GIFT_E_INVAL;
    if ((uintptr_t)aad16 & 15) return GIFT_E_ALIGN;
    c->aad = aad16;
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

uint32_t gift_version(void) { return GIFT_VERSION; }

uint64_t gift_launch_count(const gift_ctx* c) { return c ? c->launches : 0; }

}  // extern "C"

// ---------------------------------------------------------------------------
// gift_seg_encrypt_static: the export call for callers that must not allocate
// ---------------------------------------------------------------------------
//
// Same kernels as gift_seg_encrypt, but the per-call scratch (work list, partial
// hashes, tickets, counters) lives in one file-scope device array instead of
// memory the ctx grows with cudaMalloc.  The array belongs to the loaded library:
// every GPU that loads libgift.so holds GIFT_STATIC_SCRATCH_BYTES of it until the
// process exits, and every call on that GPU shares it.

#define GIFT_STATIC_MAX_SEGS 65536u

namespace {

constexpr size_t STATIC_OFF_PREFIX = 256;                                                   // after Globals
constexpr size_t STATIC_OFF_ACC = STATIC_OFF_PREFIX + ((size_t)GIFT_STATIC_MAX_SEGS + 64) * 8;   // 16-byte aligned
constexpr size_t STATIC_OFF_TICKET = STATIC_OFF_ACC + (size_t)GIFT_STATIC_MAX_SEGS * 16;
constexpr size_t STATIC_SCRATCH_BYTES = STATIC_OFF_TICKET + (size_t)GIFT_STATIC_MAX_SEGS * 4;
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
    if (!c || !segs || !tags_out || !status) return nseg == 0 && c ? GIFT_OK : GIFT_E_INVAL;
    if (nseg == 0) return GIFT_OK;
    if (nseg > GIFT_STATIC_MAX_SEGS) return GIFT_E_RANGE;     // larger tables need gift_seg_encrypt
    if (!src || !dst) return GIFT_E_INVAL;
    if (((uintptr_t)src & 15) || ((uintptr_t)dst & 15) || ((uintptr_t)tags_out & 15)) return GIFT_E_ALIGN;
    if (pages && (!pages->table || pages->page_bytes == 0)) return GIFT_E_INVAL;
    if (pages && (pages->page_bytes & 15)) return GIFT_E_ALIGN;
    if (labels && (!labels->owner_map || (!pages && labels->unit_bytes == 0))) return GIFT_E_INVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    unsigned char* scratch = nullptr;
    const int rc0 = static_scratch_for(c->device, &scratch);
    if (rc0 != GIFT_OK) return rc0;
    cudaStream_t st = (cudaStream_t)stream;

    CallArgs a;
    memset(&a, 0, sizeof(a));
    a.src = (const uint8_t*)src;
    a.dst = (uint8_t*)dst;
    a.buf_bytes = buf_bytes;
    a.segs = segs;
    a.nseg = nseg;
    if (pages) { a.page_table = pages->table; a.n_pages = pages->n; a.page_bytes = pages->page_bytes; }
    if (labels) { a.owner_map = labels->owner_map; a.n_units = labels->n_units; a.unit_bytes = labels->unit_bytes; }
    a.tags = tags_out;
    a.status = status;
    a.hot = c->d_hot;
    a.pow = c->d_pow;
    a.max_users = c->max_users;
    a.glob = reinterpret_cast<Globals*>(scratch);
    a.wprefix = reinterpret_cast<unsigned long long*>(scratch + STATIC_OFF_PREFIX);
    a.acc = reinterpret_cast<uint4*>(scratch + STATIC_OFF_ACC);
    a.ticket = reinterpret_cast<uint32_t*>(scratch + STATIC_OFF_TICKET);
    a.resident_warps = (uint32_t)c->num_sms * (uint32_t)(c->threads / 32);

    // The array still holds the previous call's values: the counters are cleared here, the
    // per-segment accumulators and tickets by the plan kernel, the weight prefix by the scan kernel.
    CU_TRY(cudaMemsetAsync(a.glob, 0, sizeof(Globals), st));
    plan_kernel<MODE_ENCRYPT><<<(nseg + 7) / 8, 256, 0, st>>>(a);
    scan_kernel<<<1, 1024, 0, st>>>(a);
    c->launches += 2;
    const int rc = launch_crypt<MODE_ENCRYPT>(c, a, st);
    if (rc != GIFT_OK) return rc;
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}

