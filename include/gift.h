/*
 * libgift: per-user encryption of ownership-segmented GPU buffers, with the
 * ownership-label check and segment-level flow rules, for one NVIDIA B200.
 *
 * The library realises the data path of the paper's encryption-as-isolation scheme
 * (paper sec. 3, workflow steps 0 and 3-6): every user datum that leaves the
 * protected domain is ciphertext under its owner's key, and data entering it
 * is decrypted with the key of the owner the untrusted framework claims, so a
 * false claim ends in a decryption failure instead of a leak.  The paper names
 * no cipher; this library uses AES-128-GCM per segment (AES-128 in counter
 * mode, FIPS-197 / SP 800-38A, with the GHASH tag of SP 800-38D, 96-bit IV,
 * 128-bit tag, empty AAD).  The tag is what makes a wrong owner or a tampered
 * byte detectable.
 *
 * Conventions common to all calls
 *  - Every call returns an int: GIFT_OK (0) or a negative GIFT_E_* code for an
 *    error detected synchronously on the host (bad argument, CUDA error).
 *    What happens to one segment never comes back as the return code; it is
 *    written to the device array status[] as a bit set of GIFT_ST_* flags.
 *  - Unless stated otherwise every data pointer is a DEVICE pointer owned by
 *    the caller, valid on the ctx's device.  The ctx owns only key material,
 *    tables and scratch, and overwrites key material with zeros on destroy.
 *  - Calls enqueue work on the given stream (a cudaStream_t passed as void*;
 *    NULL is the default stream) and do not wait for it.  The exception is
 *    scratch growth: a call whose segment count exceeds what the ctx has seen
 *    so far (see gift_ctx_reserve) reallocates scratch, which synchronises.
 *  - gift_pages, gift_labels and gift_rule are small HOST structures that carry device
 *    pointers; they are read during the call and need not outlive it.
 *  - A ctx must not be used from two threads, or on two streams, at once (the
 *    host-boundary calls say what they allow).
 *  - Ownership labels are int32: a user id >= 0, GIFT_OWNER_PARAM for model
 *    parameters (paper sec. 4.2 gives parameters an owner id of their own),
 *    GIFT_OWNER_NONE for memory no record covers (sec. 4.2, unowned memory may
 *    not be read), GIFT_OWNER_CONFLICT for an output whose sources disagree.
 */
#ifndef GIFT_H
#define GIFT_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GIFT_OK          0
#define GIFT_E_INVAL    (-1)   /* null / inconsistent argument */
#define GIFT_E_NOMEM    (-2)   /* host or device allocation failed */
#define GIFT_E_CUDA     (-3)   /* a CUDA runtime call failed */
#define GIFT_E_RANGE    (-4)   /* user id outside [0, max_users), size over a stated limit */
#define GIFT_E_ALIGN    (-5)   /* buffer or page size not 16-byte aligned */

#define GIFT_ST_TAG_MISMATCH    1u   /* decrypt/verify: tag does not match (tampered, or wrong owner claimed) */
#define GIFT_ST_OWNER_MISMATCH  2u   /* encrypt: a covered unit is owned by someone else, or by PARAM */
#define GIFT_ST_UNOWNED         4u   /* encrypt: a covered unit is NONE or CONFLICT */
#define GIFT_ST_NO_KEY          8u   /* the owner has no key in the ctx */
#define GIFT_ST_BAD_DESC       16u   /* descriptor misaligned, out of range, or reserved flags set */
#define GIFT_ST_OVERLAP        32u   /* shares bytes with another segment of the call (only with GIFT_CTX_CHECK_OVERLAP) */

#define GIFT_OWNER_PARAM     (-1)
#define GIFT_OWNER_NONE      (-2)
#define GIFT_OWNER_CONFLICT  (-3)

/* Longest segment: the GCM limit of 2^36 - 32 bytes. */
#define GIFT_MAX_SEG_BYTES  ((((uint64_t)1) << 36) - 32)

typedef struct gift_ctx gift_ctx;

/* One ownership segment: a contiguous same-owner region (paper sec. 4.1,
 * insight 1, and sec. 4.2 on the granularity of records).  40 bytes; a device array.
 *   owner  the owner the caller claims for the segment (selects the key)
 *   flags  reserved, must be 0
 *   offset flat mode: byte offset of the segment in the buffer, multiple of 16
 *   len    payload bytes, 0 <= len <= GIFT_MAX_SEG_BYTES, any value (the last
 *          cipher block may be partial; len 0 yields the tag of the empty message)
 *   nonce  the 96-bit IV; unique per (key, encryption) - the library never
 *          invents or checks nonces
 *   page0  paged mode: index of the segment's first entry in the page table */
typedef struct {
    int32_t  owner;
    uint32_t flags;
    uint64_t offset;
    uint64_t len;
    uint8_t  nonce[12];
    uint32_t page0;
} gift_seg;

/* Paged mode (block-table indexed KV cache, paper sec. 4.2): byte k of a
 * segment lives at table[page0 + k / page_bytes] * page_bytes + k % page_bytes
 * of the buffer.  table is a device array of n physical page numbers;
 * page_bytes is a positive multiple of 16.  Pass NULL for flat mode. */
typedef struct {
    const int32_t* table;
    uint32_t       n;
    uint64_t       page_bytes;
} gift_pages;

/* Ownership records of the buffer: owner_map[u] is the label of unit u (device
 * array of n_units labels).  Flat mode: unit u covers bytes [u*unit_bytes,
 * (u+1)*unit_bytes); a segment covers every unit its byte range touches.
 * Paged mode: one unit per physical page, unit_bytes ignored.  An empty
 * segment covers no unit.  Pass NULL to skip label handling. */
typedef struct {
    int32_t* owner_map;
    uint32_t n_units;
    uint64_t unit_bytes;
} gift_labels;

/* Create a context on CUDA device `device` able to hold keys for user ids
 * 0 .. max_users-1 (about 17 KiB of device memory per user: round keys and
 * powers of the hash subkey), max_users <= 2^20.  flags is 0 or a set of
 *   GIFT_CTX_TWO_TABLES     the cipher kernel keeps two AES tables (64 KiB of shared memory
 *                           per SM) instead of four (128 KiB): a few per cent slower, for
 *                           callers whose own kernels must share the SM
 *   GIFT_CTX_CHECK_OVERLAP  every segment call first checks that the segments of its table
 *                           occupy distinct memory (paper sec. 4.3, rule step 3; sec. 3 step 4:
 *                           every byte has one owner).  A segment that shares a byte with
 *                           another valid segment of the call, or that names one physical page
 *                           twice, is refused like a bad descriptor: status GIFT_ST_OVERLAP,
 *                           nothing of it read or written, tag zero on encrypt.  Empty segments
 *                           and segments with a bad descriptor take no part.  Costs one more
 *                           launch per call: all pairs for flat tables (at most 65 536
 *                           segments, else GIFT_E_RANGE), one claim per physical page for paged
 *                           ones.  Without the flag overlapping segments give undefined bytes.
 *   GIFT_CTX_SPLIT_LAUNCH   never use the single-launch form that small tables take (for
 *                           measurements; results are the same)
 * Host call; synchronises. */
#define GIFT_CTX_TWO_TABLES     1u
#define GIFT_CTX_CHECK_OVERLAP  2u
#define GIFT_CTX_SPLIT_LAUNCH   4u
int gift_ctx_create(gift_ctx** out, int device, uint32_t max_users, uint32_t flags);

/* Zero all key material on the device and free the ctx.  Synchronises. */
int gift_ctx_destroy(gift_ctx* ctx);

/* Pre-size the per-call scratch (work list, partial hashes) for calls of up to
 * max_segs segments so that later calls never reallocate.  Synchronises. */
int gift_ctx_reserve(gift_ctx* ctx, uint32_t max_segs);

/* Install keys (paper sec. 3 step 0: the monitor stores user-specific keys in
 * its protected memory).  user_ids[n] and keys16[n*16] are HOST arrays; key i
 * belongs to user user_ids[i] in [0, max_users).  The expanded round keys, the
 * hash subkey H = E_K(0) and its powers are derived on the device.  The host
 * staging copy is wiped before the call returns. */
int gift_set_keys(gift_ctx* ctx, const int32_t* user_ids, const uint8_t* keys16, uint32_t n,
                  void* stream);

/* Remove users' keys (device material overwritten with zeros). */
int gift_clear_keys(gift_ctx* ctx, const int32_t* user_ids, uint32_t n, void* stream);

/* Export (paper sec. 3 steps 5-6; sec. 4.1: the key is selected from the
 * ownership state, not from the framework's claim).  For every segment, in any
 * order: if labels are given, every covered unit must carry the segment's
 * owner; the owner must have a key.  Then dst receives AES-128-CTR ciphertext
 * of src (counter blocks nonce || BE32(2), BE32(3), ...) and tags_out[i] the
 * 16-byte GCM tag.  Otherwise the segment's dst bytes are left as they were,
 * its tag is 16 zero bytes and status[i] says why.  src may equal dst; bytes
 * outside all segments are never written.  Segments of one call must not
 * overlap (GIFT_CTX_CHECK_OVERLAP makes the call check it).  A table of at most
 * 1024 segments runs as a single kernel launch.  buf_bytes is the size of src
 * and of dst.  src and dst are addresses the device can dereference: device
 * memory, or page-locked host memory mapped into the device's address space
 * (the boundary copy of sec. 4.5 fused into the cipher: the kernel then reads
 * or writes across the bus itself). */
int gift_seg_encrypt(gift_ctx* ctx, const void* src, void* dst, uint64_t buf_bytes,
                     const gift_seg* segs, uint32_t nseg, const gift_pages* pages,
                     const gift_labels* labels, uint8_t* tags_out, uint32_t* status, void* stream);

/* gift_seg_encrypt for callers that are not allowed to allocate device memory (the paper
 * has no counterpart; it is an addition of this library).  Some hosts of this code cannot
 * call cudaMalloc at the point where they export data: a serving loop that has handed all
 * device memory to its own pool, a plugin that runs under a framework's allocator, code
 * that runs where an allocation would stall every stream.  gift_seg_encrypt grows its
 * scratch with cudaMalloc when a call has more segments than any before it; this entry
 * point never does.  It calls no cudaMalloc, cudaFree or other allocating routine: its
 * scratch (work list, partial hashes, counters) is a fixed array inside the library image,
 * about 2 MB, which every GPU that loads the library holds until the process exits.
 *   - Arguments, results and status words are exactly those of gift_seg_encrypt, bound AAD
 *     included; the ctx (created earlier, when allocation was still allowed) supplies the
 *     keys.  On a ctx with GIFT_CTX_CHECK_OVERLAP only flat tables are taken (the check of
 *     paged tables needs memory that grows with the buffer): GIFT_E_INVAL otherwise.
 *   - nseg must not exceed GIFT_STATIC_MAX_SEGS (65536); a larger table is refused with
 *     GIFT_E_RANGE and nothing is launched.
 *   - The first call on a device looks up the array's device address; make that first
 *     call before any stream capture begins.
 *   - All calls on one GPU share the array.  Each call clears what it needs, so calls may
 *     follow one another freely on one stream, but two calls whose kernels can overlap on
 *     the GPU (different streams, different ctxs, different threads) race on it and give
 *     wrong tags.  Serialise them, or use gift_seg_encrypt for the concurrent ones. */
#define GIFT_STATIC_MAX_SEGS 65536u
int gift_seg_encrypt_static(gift_ctx* ctx, const void* src, void* dst, uint64_t buf_bytes,
                            const gift_seg* segs, uint32_t nseg, const gift_pages* pages,
                            const gift_labels* labels, uint8_t* tags_out, uint32_t* status, void* stream);

/* Bind additional authenticated data to the tags (no counterpart in the paper; the AAD of
 * SP 800-38D).  After this call gift_seg_encrypt, gift_seg_encrypt_static, gift_seg_decrypt,
 * gift_verify_tags and the host-boundary calls authenticate the 16 bytes
 * aad16[16*i .. 16*i+15] (device array of n entries, 16-byte aligned) together with segment i
 * of the call's table: a tag then also vouches for, say, (owner, logical position, epoch), so
 * that a ciphertext block presented under the right key and nonce but in the wrong role fails
 * verification.  A call with more than n segments is refused with GIFT_E_RANGE.  NULL (the
 * initial state) turns binding off.  The pointer is used by the calls that follow, not
 * copied. */
int gift_ctx_bind_aad(gift_ctx* ctx, const uint8_t* aad16, uint32_t n);

/* Import (paper sec. 3 steps 3-4): decrypt each segment with the CLAIMED
 * owner's key after checking tags_in[i] over the received ciphertext.  On a
 * match dst receives the plaintext and, if labels are given, the covered units
 * are recorded as owned by the claimed owner.  On a mismatch, or when the
 * claimed owner has no key, the segment's dst bytes are all zero and the
 * covered units become GIFT_OWNER_NONE (a unit covered by both a good and a
 * failed segment ends up NONE).  BAD_DESC and OVERLAP segments touch nothing. */
int gift_seg_decrypt(gift_ctx* ctx, const void* src, void* dst, uint64_t buf_bytes,
                     const gift_seg* segs, uint32_t nseg, const gift_pages* pages,
                     gift_labels* labels, const uint8_t* tags_in, uint32_t* status, void* stream);

/* Tag check only: status[i] as gift_seg_decrypt would set it; nothing else is written. */
int gift_verify_tags(gift_ctx* ctx, const void* src, uint64_t buf_bytes, const gift_seg* segs,
                     uint32_t nseg, const gift_pages* pages, const uint8_t* tags_in,
                     uint32_t* status, void* stream);

/* Token mode (paper sec. 4.5, the paragraph on tokens): each token is encrypted on its own
 * with a block cipher, not as part of a stream, because the framework splits and appends
 * sequences; a 64-bit token is extended to 128 bits with a 64-bit nonce so that equal
 * tokens give different ciphertexts, and the end-of-sequence token gets a special
 * ciphertext that tells the framework that generation is complete.
 * Here: block = LE64(token) || LE64(nonce), AES-128 under the key of owners[i]; a token
 * equal to eos_token is replaced by the public marker of 16 bytes 0xFF.  tokens, nonces,
 * owners (device arrays of n) give out16 (n x 16 bytes, 16-byte aligned) and status[i]
 * (0, or GIFT_ST_NO_KEY with a zero block).  There is no integrity tag in this mode:
 * decrypting under a wrong owner yields another token, never the plaintext. */
int gift_tok_encrypt(gift_ctx* ctx, const uint64_t* tokens, const uint64_t* nonces, const int32_t* owners,
                     uint32_t n, uint64_t eos_token, uint8_t* out16, uint32_t* status, void* stream);

/* Inverse of gift_tok_encrypt with the CLAIMED owners (FIPS-197 inverse cipher): the nonce
 * is dropped (nonces_out may be NULL), the marker decrypts to eos_token, a claimed owner
 * without a key gives token 0 and GIFT_ST_NO_KEY. */
int gift_tok_decrypt(gift_ctx* ctx, const uint8_t* in16, const int32_t* owners, uint32_t n, uint64_t eos_token,
                     uint64_t* tokens_out, uint64_t* nonces_out, uint32_t* status, void* stream);

/* A flow rule (paper sec. 4.3, rule generation, steps 4 and 5): for
 * every output unit, its non-parameter sources must share one owner, which the
 * output receives; operands declared as parameters must be labelled PARAM.
 * The join treats PARAM as neutral, equal users as that user, and anything
 * else (different users, NONE, CONFLICT) as CONFLICT.
 *   GIFT_RULE_IDENTITY   out[j] = in0[j]                       (copies, swaps)
 *   GIFT_RULE_ROWWISE    out[j] = join over row operands k of in_k[j]; operand
 *                        k with bit k of param_mask set is a one-unit map that
 *                        must equal PARAM, else every out[j] is CONFLICT
 *                        (AddBias, AddResidual, FindMax, MatrixMultiply)
 *   GIFT_RULE_SEGREDUCE  for reduction segment s (a request): m = join of
 *                        in0[t] for t in [seg_ptr[s], seg_ptr[s+1]) and of
 *                        in1[src_idx[e]] for e in [src_ptr[s], src_ptr[s+1]);
 *                        out[t] = m for the segment's t (decoding-stage
 *                        attention over a block table, paper sec. 7.2); an
 *                        out-of-range src_idx counts as NONE; outputs no
 *                        segment covers are CONFLICT
 *   GIFT_RULE_BROADCAST  out[j] = in0[gather[j]]; out-of-range gather gives CONFLICT
 * n_in is the number of input maps (ROWWISE: 1..8; SEGREDUCE: 2; others: 1),
 * n_in0 the length of in0 (BROADCAST), n_in1 the length of in1 and n_src the length of
 * src_idx (SEGREDUCE).  All index arrays are device arrays supplied by the untrusted
 * framework, so nothing in them is trusted: seg_ptr and src_ptr (n_seg + 1 entries each)
 * must be valid CSR pointers (first entry >= 0, non-decreasing, last entry <= n_out and
 * <= n_src); if they are not, the launch as a whole is rejected: every out[j] is CONFLICT. */
#define GIFT_RULE_IDENTITY   0u
#define GIFT_RULE_ROWWISE    1u
#define GIFT_RULE_SEGREDUCE  2u
#define GIFT_RULE_BROADCAST  3u

typedef struct {
    uint32_t kind;
    uint32_t n_out;
    uint32_t n_in;
    uint32_t n_seg;
    uint32_t n_in0;
    uint32_t n_in1;
    uint32_t n_src;
    const int32_t* seg_ptr;
    const int32_t* src_ptr;
    const int32_t* src_idx;
    const int32_t* gather;
    uint32_t param_mask;
} gift_rule;

/* Apply one rule on the device.  rule and in_owner_maps are HOST structures
 * (an array of n_in device pointers).  out_owner_map may alias an input: the
 * rule reads a snapshot.  viol[0] receives the number of CONFLICT outputs and
 * viol[1] the smallest such index (0xFFFFFFFF if none).  The paper rejects the
 * launch on any violation (sec. 4.1, insight 3); here out is always written
 * and committing it is the caller's decision. */
int gift_propagate_labels(gift_ctx* ctx, const gift_rule* rule, const int32_t* const* in_owner_maps,
                          int32_t* out_owner_map, uint32_t* viol, void* stream);

/* The rules of consecutive kernels applied in one launch (paper sec. 4.3 runs the rule of
 * every kernel of a forward pass; a label map is a few hundred KiB, so a rule on its own
 * costs only its launch).  Rule k is rules[k] with inputs in_owner_maps[k] (HOST array of
 * its n_in device pointers) and output out_owner_maps[k]; it sees everything rules 0..k-1
 * wrote, exactly as n_rules calls of gift_propagate_labels in that order would.  viol is a
 * device array of 2*n_rules words: viol[2k] the number of CONFLICT outputs of rule k and
 * viol[2k+1] the smallest such index (0xFFFFFFFF if none).  n_rules <= GIFT_CHAIN_MAX, else
 * GIFT_E_RANGE.  Unlike gift_propagate_labels the chain takes no snapshot: a rule's output
 * must not overlap the map it gathers from (BROADCAST in0, SEGREDUCE in1), else
 * GIFT_E_INVAL; writing a map in place at the same index (IDENTITY, ROWWISE, SEGREDUCE
 * in0) is fine; the index arrays must not be outputs of the chain.  One launch of a single
 * thread-block cluster (16 CTAs where the device can co-schedule them, else 8): meant for
 * maps of up to a few million units. */
#define GIFT_CHAIN_MAX 8u
int gift_propagate_chain(gift_ctx* ctx, const gift_rule* rules, const int32_t* const* const* in_owner_maps,
                         int32_t* const* out_owner_maps, uint32_t n_rules, uint32_t* viol, void* stream);

/* Multi-stream launch-order check (paper sec. 4.4, concurrency control): the ownership
 * record of a segment is extended with its last writer kernel and last reader kernels, each
 * a (stream, sequence) pair, and a kernel counts as completed once a synchronisation of its
 * stream follows its launch.  A reader of M may launch only if M's last writer, when on
 * another stream, has completed; a writer of M only if M's last readers and last writer on
 * other streams have completed.  This call checks a whole recorded trace at once.
 *   kind[e]    0 kernel launch, 1 synchronisation of stream[e]      (device, n_events)
 *   stream[e]  stream id in [0, n_streams), n_streams <= 32         (device, n_events)
 *   seg_ptr / seg_event / seg_write: for every memory segment, the launches that access
 *   it in launch order (the history its record accumulates): event index and 0 read /
 *   1 write (device; seg_ptr has n_segments + 1 entries).  A launch that reads and writes
 *   a segment appears twice, adjacent.
 * flags[e] (device, n_events) receives GIFT_RACE_* bits for every launch that breaks an
 * invariant (the monitor would have held it back); the records advance as if it had run.
 * summary[0] = number of flagged launches, summary[1] = first flagged event or 0xFFFFFFFF.
 * The struct is host memory; the call may grow a scratch array (synchronises then). */
#define GIFT_RACE_RAW 1u   /* reads a segment whose last writer on another stream is in flight */
#define GIFT_RACE_WAR 2u   /* writes a segment that a reader on another stream may still read */
#define GIFT_RACE_WAW 4u   /* writes a segment whose last writer on another stream is in flight */
typedef struct {
    uint32_t n_events, n_streams, n_segments;
    const uint8_t* kind;
    const int32_t* stream;
    const int32_t* seg_ptr;
    const int32_t* seg_event;
    const uint8_t* seg_write;
} gift_trace;
int gift_check_launch_order(gift_ctx* ctx, const gift_trace* trace, uint32_t* flags, uint32_t* summary,
                            void* stream);

/* Two-level ownership index (paper sec. 4.2, the ownership data structure): the first level
 * maps a base address to a tensor record (base address, shape, element size and the
 * ownership-related dimensions, e.g. (0) for the rows of a matrix or (0,1,3) of a
 * 5-dimensional KV tensor); the second level maps the subscripts of those dimensions to an
 * owner.  A record is host memory; `owners` is a device array with one label per
 * combination of ownership-related subscripts, row-major. */
#define GIFT_MAX_DIMS 5
typedef struct {
    uint64_t base;
    uint32_t ndim, elem_size;
    uint64_t shape[GIFT_MAX_DIMS];
    uint32_t odim_mask;              /* bit d set: dimension d decides ownership */
    const int32_t* owners;
} gift_tensor_rec;

/* One tensor argument of a kernel launch as the framework presents it.  Arguments that
 * carry the same non-zero alias_group are meant to alias (the alias nodes of the paper's flow-graph figure). */
typedef struct {
    uint64_t base;
    uint32_t ndim, alias_group;
    uint64_t shape[GIFT_MAX_DIMS];
} gift_kernel_arg;

#define GIFT_ARG_OK       0u
#define GIFT_ARG_UNKNOWN  1u   /* no record at this base address: memory the monitor does not know (sec. 4.2) */
#define GIFT_ARG_SHAPE    2u   /* argument shape differs from the record */
#define GIFT_ARG_ALIAS    4u   /* overlaps another argument without being declared an alias */

/* Steps (1)-(3) of a flow rule (paper sec. 4.3): find each argument's record by base
 * address, compare shapes, detect unintended aliasing.  Pure host call on host arrays;
 * rec_of_arg[i] is the record index or -1, arg_status[i] a set of GIFT_ARG_* bits. */
int gift_resolve_args(const gift_tensor_rec* recs, uint32_t n_rec, const gift_kernel_arg* args, uint32_t n_args,
                      int32_t* rec_of_arg, uint32_t* arg_status);

/* The contiguous runs of the slice [lo[d], hi[d]) of a recorded tensor (an ownership slice
 * such as C[1,2,:,0:8,:]), expressed as page numbers in units of the run length counted
 * from the tensor's base: a paged segment with page_bytes = *run_bytes and these table
 * entries covers exactly the slice, in row-major order.  Pure host call.  table may be NULL
 * to query *run_bytes and *n_runs.  GIFT_E_ALIGN when the run length is not a multiple of
 * 16 bytes or a run does not start on a multiple of it. */
int gift_slice_runs(const gift_tensor_rec* rec, const uint64_t* lo, const uint64_t* hi, uint64_t* run_bytes,
                    uint32_t* n_runs, int32_t* table, uint32_t table_cap);

/* Expand the level-2 records of a tensor into one label per run of run_bytes bytes
 * (unit_owner, device, n_units = tensor bytes / run_bytes): the owner map that the paged
 * segment calls take.  A run that spans several records (eight slots of a block whose
 * records are per slot) gets the label they agree on, or GIFT_OWNER_CONFLICT; a run that
 * is neither a part of one record nor a whole number of records gives GIFT_E_ALIGN. */
int gift_expand_owners(gift_ctx* ctx, const gift_tensor_rec* rec, uint64_t run_bytes, int32_t* unit_owner,
                       uint32_t n_units, void* stream);

/* Secure swap space (paper sec. 4.5): KV blocks swapped into the monitor's own memory need
 * no encryption, but their ownership records must survive the round trip.  swap_out saves
 * the labels of the listed units
 * (saved[i] = owner_map[units[i]]) and marks the units GIFT_OWNER_NONE, so that the freed
 * slots cannot be read; swap_in writes the saved labels to the units the blocks return to,
 * which need not be the ones they left.  A unit index out of range, or a swap-in onto a
 * unit that is still owned (it becomes GIFT_OWNER_CONFLICT), is counted in viol[0] with the
 * smallest offending list position in viol[1] (0xFFFFFFFF if none).  The listed units of
 * one call must be distinct.  All arrays are device arrays. */
int gift_labels_swap_out(gift_ctx* ctx, int32_t* owner_map, uint32_t n_units, const int32_t* units, uint32_t n,
                         int32_t* saved, uint32_t* viol, void* stream);
int gift_labels_swap_in(gift_ctx* ctx, int32_t* owner_map, uint32_t n_units, const int32_t* units, uint32_t n,
                        const int32_t* saved, uint32_t* viol, void* stream);

/* Text for a GIFT_E_* code; never NULL. */
const char* gift_strerror(int code);

/* For a call that returned GIFT_E_CUDA or GIFT_E_NOMEM: the CUDA runtime's name for the
 * error and where in the library it was met, as text; the last such failure of the calling
 * thread ("" if none).  Never NULL. */
const char* gift_last_error_detail(void);

/* Library version, major*10000 + minor*100 + patch. */
uint32_t gift_version(void);

/* Number of this library's kernels launched through the ctx since creation. */
uint64_t gift_launch_count(const gift_ctx* ctx);

/* Device timing of the segment-cipher kernel (diagnostics; no paper counterpart).  While
 * enabled, every gift_seg_encrypt / decrypt / verify call brackets its cipher kernel with
 * CUDA events on the call's stream.  gift_timing_read waits for the recorded events,
 * returns their summed duration in milliseconds and the number of launches since the last
 * read, and resets both.  At most 1024 launches are kept between reads. */
int gift_timing_enable(gift_ctx* ctx, int on);
int gift_timing_read(gift_ctx* ctx, double* total_ms, uint32_t* launches);

/* Host-boundary calls (paper sec. 4.5, the swap path of KV blocks, and sec. 5, the bounce
 * copy between host and device): export to, and import from, page-locked HOST memory with
 * the copies fused into the call.  The table is cut into chunks (HOST array): chunk k holds
 * the segments [seg_lo, seg_hi) of the table, all of whose bytes lie in the byte range
 * [byte_lo, byte_hi) of the buffer; chunks must not share segments or bytes.  Chunk k runs on
 * one of three streams the ctx owns, each with its own scratch, so that the upload of one
 * chunk, the cipher of the previous one and the download of the one before overlap and both
 * bus directions stay busy.  The work is ordered after what `stream` holds at the time of
 * the call, and `stream` waits for all of it; the call itself returns without waiting.
 * Copies are plain cudaMemcpyAsync, one per chunk and direction.  byte_lo and byte_hi are
 * multiples of 16.  Consecutive calls may be given different streams (and their own staging
 * and host buffers) so that the download of one overlaps the upload of the next; they must
 * still be issued from one thread.  With GIFT_CTX_CHECK_OVERLAP the check covers the segments
 * of one chunk at a time, and all chunks run on one internal stream. */
typedef struct {
    uint64_t byte_lo, byte_hi;
    uint32_t seg_lo, seg_hi;
} gift_chunk;

/* Export.  Per chunk: upload h_src[byte range] into d_plain (skipped when h_src is NULL: the
 * plaintext is already in d_plain), clear d_cipher[byte range], encrypt the chunk's segments
 * out of place from d_plain into d_cipher exactly as gift_seg_encrypt would (labels, status
 * words, tags), download d_cipher[byte range] to h_dst, the chunk's tags to h_tags and its
 * status words to h_status.  Only ciphertext leaves the device: bytes of the range that no
 * accepted segment covers, a refused segment's bytes among them, arrive in h_dst as zeros.
 * d_plain is left unchanged.  h_src (or NULL), h_dst, h_tags (nseg x 16) and h_status (nseg)
 * are page-locked host memory; d_plain, d_cipher (buf_bytes each, distinct), segs, d_tags,
 * d_status are device memory.  GIFT_E_INVAL if a chunk is out of range or empty of order
 * (seg_lo > seg_hi, byte_lo > byte_hi). */
int gift_export_to_host(gift_ctx* ctx, const void* h_src, void* h_dst, void* d_plain, void* d_cipher,
                        uint64_t buf_bytes, const gift_seg* segs, uint32_t nseg, const gift_chunk* chunks,
                        uint32_t n_chunks, const gift_pages* pages, const gift_labels* labels, uint8_t* d_tags,
                        uint32_t* d_status, uint8_t* h_tags, uint32_t* h_status, void* stream);

/* Import.  Per chunk: upload the ciphertext h_src[byte range] into d_buf and the chunk's
 * tags from h_tags into d_tags, decrypt in place exactly as gift_seg_decrypt would (failed
 * segments zero-filled, labels written), download the chunk's status words to h_status.  The
 * plaintext stays on the device. */
int gift_import_from_host(gift_ctx* ctx, const void* h_src, const uint8_t* h_tags, void* d_buf, uint64_t buf_bytes,
                          const gift_seg* segs, uint32_t nseg, const gift_chunk* chunks, uint32_t n_chunks,
                          const gift_pages* pages, gift_labels* labels, uint8_t* d_tags, uint32_t* d_status,
                          uint32_t* h_status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GIFT_H */
