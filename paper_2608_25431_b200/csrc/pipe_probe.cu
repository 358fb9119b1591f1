// Issue-rate probes for the integer, multiply and shared-memory pipes of one SM.
//
// The segment cipher is bound by integer instruction throughput, so its roofline
// needs the per-SM rates of the instructions it is made of.  Each probe runs
// 1024 threads per SM over long unrolled chains of one instruction kind (eight
// independent chains per thread hide the latency), times the loop with the SM
// cycle counter and reports lane-operations per SM clock.
//
// Diagnostics only: built into libgift_probe.so, not into libgift.so, and not declared in
// the public header.  Entry point:
//   int gift_probe_pipe(int device, int kind, uint32_t iters, double* lane_ops_per_clk_per_sm, double* sm_mhz)
// kind: 0 three-input logic, 1 32x32+64 wide multiply-add, 2 byte permute, 3 conflict-free
// shared-memory load, 4 funnel shift, 5 integer add, 6 logic and wide multiply interleaved,
// 7 32-bit multiply-add, 8 logic and shared loads interleaved, 9-19 further kinds and
// pairings, 20-32 instruction mixes like the first cipher kernel's, 33 bit reversal, 34 logic
// and bit reversal, 35 the single-bit tensor-core product mma.sync m16n8k128 (and, popcount),
// 36 two 32-bit multiply-adds feeding one logic operation.  Returns 0, or a negative code
// (-1 bad argument, -3 CUDA error).  Host call; allocates a few KB, synchronises.
#include <cuda_runtime.h>
#include <stdint.h>

#define GIFT_OK 0
#define GIFT_E_INVAL (-1)
#define GIFT_E_NOMEM (-2)
#define GIFT_E_CUDA (-3)
#define GIFT_E_RANGE (-4)

namespace {

constexpr int CHAINS = 8;
constexpr int UNROLL = 32;

template <int KIND>
__global__ void __launch_bounds__(1024, 1) probe_kernel(uint32_t iters, uint32_t seed, unsigned long long* cycles,
                                                        uint32_t* sink)
{
    // tab[i] is a multiple of 32 below 2048, so tab[tab[i] + lane] stays inside the table and
    // every lane of a warp reads its own bank
    __shared__ uint32_t tab[2048];
    for (int i = threadIdx.x; i < 2048; i += blockDim.x) tab[i] = ((i >> 5) * 37u + seed) & 2047u & ~31u;
    __syncthreads();
    const volatile uint32_t* vtab = tab;
    uint32_t x[CHAINS], y[CHAINS];
    unsigned long long w[CHAINS];
#pragma unroll
    for (int c = 0; c < CHAINS; c++) {
        x[c] = seed * (c + 1) + threadIdx.x;
        y[c] = seed + c;
        if (KIND == 3) x[c] = (x[c] & 2047u & ~31u);
        w[c] = x[c];
    }
    const uint32_t k1 = seed | 1u, k2 = seed * 3u + 5u;
    const uint32_t lane4 = (threadIdx.x & 31u);
    __syncthreads();
    const long long t0 = clock64();
    for (uint32_t it = 0; it < iters; it++) {
#pragma unroll
        for (int u = 0; u < UNROLL; u++) {
#pragma unroll
            for (int c = 0; c < CHAINS; c++) {
                if (KIND == 0) {          // three-input logic
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k2));
                } else if (KIND == 1) {   // 32x32+64 -> 64 multiply-add
                    asm volatile("mad.wide.u32 %0, %1, %2, %0;" : "+l"(w[c]) : "r"(x[c]), "r"(k1));
                } else if (KIND == 2) {   // byte permute
                    asm volatile("prmt.b32 %0, %0, %1, 0x2103;" : "+r"(x[c]) : "r"(k1));
                } else if (KIND == 3) {   // conflict-free shared-memory load, address from the previous load
                    x[c] = vtab[x[c] + lane4];
                } else if (KIND == 4) {   // funnel shift
                    asm volatile("shf.l.wrap.b32 %0, %0, %1, 7;" : "+r"(x[c]) : "r"(k1));
                } else if (KIND == 5) {   // three-input add
                    asm volatile("add.u32 %0, %0, %1;" : "+r"(x[c]) : "r"(k1));
                } else if (KIND == 6) {   // logic and wide multiply interleaved: do they share a pipe?
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k2));
                    asm volatile("mad.wide.u32 %0, %1, %2, %0;" : "+l"(w[c]) : "r"(k2), "r"(k1));
                } else if (KIND == 7) {   // 32x32+32 -> 32 multiply-add (low half)
                    asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(x[c]) : "r"(k1), "r"(k2));
                } else if (KIND == 9) {   // 32x32 -> 64 multiply without accumulate
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                } else if (KIND == 10) {  // logic + wide multiply without accumulate
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)w[c]));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                } else if (KIND == 11) {  // logic + 32-bit multiply-add
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)w[c]));
                    asm volatile("mad.lo.u32 %0, %1, %2, %3;" : "=r"(*reinterpret_cast<uint32_t*>(&w[c])) : "r"(x[c]), "r"(k1), "r"(k2));
                } else if (KIND == 12) {  // logic + add
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)w[c]));
                    asm volatile("add.u32 %0, %1, %2;" : "=r"(*reinterpret_cast<uint32_t*>(&w[c])) : "r"(x[c]), "r"(k1));
                } else if (KIND == 13) {  // byte permute + wide multiply-add
                    asm volatile("prmt.b32 %0, %0, %1, 0x2103;" : "+r"(x[c]) : "r"(k1));
                    asm volatile("mad.wide.u32 %0, %1, %2, %0;" : "+l"(w[c]) : "r"(k2), "r"(k1));
                } else if (KIND == 14) {  // logic with an immediate operand + wide multiply-add
                    asm volatile("lop3.b32 %0, %0, %1, 0x11111111, 0x96;" : "+r"(x[c]) : "r"(k1));
                    asm volatile("mad.wide.u32 %0, %1, %2, %0;" : "+l"(w[c]) : "r"(k2), "r"(k1));
                } else if (KIND == 15) {  // two logic + one wide multiply-add
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k2));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"(k1));
                    asm volatile("mad.wide.u32 %0, %1, %2, %0;" : "+l"(w[c]) : "r"(k2), "r"(k1));
                } else if (KIND == 16) {  // shared load + wide multiply-add
                    w[c] += vtab[lane4 + (c << 5)];
                    asm volatile("mad.wide.u32 %0, %1, %2, %0;" : "+l"(w[c]) : "r"(k2), "r"(k1));
                } else if (KIND == 17) {  // logic + permute (both integer pipe)
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k2));
                    asm volatile("prmt.b32 %0, %0, %1, 0x2103;" : "+r"(x[c]) : "r"(k1));
                } else if (KIND == 18) {  // high half of a 32x32 multiply
                    asm volatile("mul.hi.u32 %0, %0, %1;" : "+r"(x[c]) : "r"(k1));
                } else if (KIND == 19) {  // logic + high-half multiply
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)w[c]));
                    asm volatile("mul.hi.u32 %0, %1, %2;" : "=r"(*reinterpret_cast<uint32_t*>(&w[c])) : "r"(x[c]), "r"(k1));
                } else if (KIND == 20) {  // the cipher kernel's mix: 11 logic, 3 wide multiplies, 2 multiply-adds, 4 lookups
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k2));
                    asm volatile("prmt.b32 %0, %0, %1, 0x2103;" : "+r"(x[c]) : "r"(k1));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"(k1));
                    x[c] ^= vtab[(x[c] & 2016u) + lane4];
                    asm volatile("prmt.b32 %0, %0, %1, 0x1032;" : "+r"(x[c]) : "r"(k2));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"((uint32_t)w[c]), "r"(k2));
                    asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(x[c]) : "r"(k1), "r"(k2));
                    asm volatile("prmt.b32 %0, %0, %1, 0x0321;" : "+r"(x[c]) : "r"(k1));
                    x[c] ^= vtab[(x[c] & 2016u) + lane4];
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k2));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"((uint32_t)(w[c] >> 32)), "r"(k1));
                    asm volatile("prmt.b32 %0, %0, %1, 0x2103;" : "+r"(x[c]) : "r"(k2));
                    x[c] ^= vtab[(x[c] & 2016u) + lane4];
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                    asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(x[c]) : "r"(k2), "r"((uint32_t)w[c]));
                    asm volatile("prmt.b32 %0, %0, %1, 0x1230;" : "+r"(x[c]) : "r"(k1));
                    x[c] ^= vtab[(x[c] & 2016u) + lane4];
                } else if (KIND == 21) {  // two logic + one wide multiply (no addend)
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)w[c]));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"((uint32_t)(w[c] >> 32)));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                } else if (KIND == 22) {  // logic + permute + wide multiply
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)w[c]));
                    asm volatile("prmt.b32 %0, %0, %1, 0x2103;" : "+r"(x[c]) : "r"((uint32_t)(w[c] >> 32)));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                } else if (KIND == 23) {  // three logic + one independent shared load
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k2));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"(k1));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k1));
                    w[c] = vtab[lane4 + (c << 5)];
                } else if (KIND == 24) {  // two logic + one multiply-add + one independent shared load
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)w[c]));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"((uint32_t)(w[c] >> 32)));
                    x[c] ^= vtab[lane4 + (c << 5)];
                } else if (KIND == 25) {  // as 21, but both logic operations read the low half of the product
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)w[c]));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"((uint32_t)w[c]));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                } else if (KIND == 26) {  // as 21, but only the high half of the product is read
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k2));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"((uint32_t)(w[c] >> 32)));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                } else if (KIND == 27) {  // two logic + one 32-bit multiply-add
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)w[c]));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"(k1));
                    asm volatile("mad.lo.u32 %0, %1, %2, %3;" : "=r"(*reinterpret_cast<uint32_t*>(&w[c])) : "r"(x[c]), "r"(k1), "r"(k2));
                } else if (KIND == 28) {  // three logic + one wide multiply
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)w[c]));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"(k1));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k1));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                } else if (KIND == 29) {  // one logic operation reads both halves of the product
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"((uint32_t)w[c]), "r"((uint32_t)(w[c] >> 32)));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"(k1));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                } else if (KIND == 30) {  // the high half goes through a multiply-add first, logic reads the copy
                    uint32_t hi2;
                    asm volatile("mad.lo.u32 %0, %1, %2, %3;" : "=r"(hi2) : "r"((uint32_t)(w[c] >> 32)), "r"(k1), "r"(k2));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(hi2));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"((uint32_t)w[c]));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                } else if (KIND == 31) {  // the high half read by a permute instead of a logic operation
                    asm volatile("prmt.b32 %0, %0, %1, 0x2143;" : "+r"(x[c]) : "r"((uint32_t)(w[c] >> 32)));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"(k1));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                } else if (KIND == 32) {  // high half read, but two independent logic operations sit between product and use
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k2));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"(k1));
                    asm volatile("mul.wide.u32 %0, %1, %2;" : "=l"(w[c]) : "r"(x[c]), "r"(k1));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k1));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x69;" : "+r"(x[c]) : "r"(k2), "r"(k2));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)(w[c] >> 32)));
                } else if (KIND == 33) {  // bit reversal
                    asm volatile("brev.b32 %0, %0;" : "+r"(x[c]));
                } else if (KIND == 34) {  // logic + bit reversal: separate pipes?
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"((uint32_t)w[c]));
                    asm volatile("brev.b32 %0, %1;" : "=r"(*reinterpret_cast<uint32_t*>(&w[c])) : "r"(x[c]));
                } else if (KIND == 35) {  // single-bit tensor-core product, 16x8x128 (and + popcount), counted as one lane-op per thread
                    uint32_t* m = reinterpret_cast<uint32_t*>(&w[c]);
                    asm volatile("mma.sync.aligned.m16n8k128.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                                 : "+r"(m[0]), "+r"(m[1]), "+r"(x[c]), "+r"(y[c]) : "r"(k1), "r"(k2), "r"(lane4));
                } else if (KIND == 36) {  // two 32-bit multiply-adds whose sum feeds one logic operation (the shipped multiply's pattern)
                    uint32_t* m = reinterpret_cast<uint32_t*>(&w[c]);
                    asm volatile("mad.lo.u32 %0, %1, %2, %3;" : "=r"(m[0]) : "r"(x[c]), "r"(k1), "r"(m[1]));
                    asm volatile("mad.lo.u32 %0, %1, %2, %3;" : "=r"(m[1]) : "r"(x[c]), "r"(k2), "r"(m[0]));
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(m[0]), "r"(m[1]));
                } else if (KIND == 8) {   // logic and shared-memory loads interleaved
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[c]) : "r"(k1), "r"(k2));
                    w[c] = vtab[lane4 + (c << 5)];
                }
            }
        }
    }
    const long long t1 = clock64();
    uint32_t acc = 0;
#pragma unroll
    for (int c = 0; c < CHAINS; c++) acc ^= x[c] ^ y[c] ^ (uint32_t)w[c] ^ (uint32_t)(w[c] >> 32);
    if (acc == 0x12345678u) sink[0] = acc;     // keeps the chains alive
    if (threadIdx.x == 0) cycles[blockIdx.x] = (unsigned long long)(t1 - t0);
}

template <int KIND>
cudaError_t run_probe(int sms, uint32_t iters, unsigned long long* d_cycles, uint32_t* d_sink, float* ms)
{
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    probe_kernel<KIND><<<sms, 1024>>>(4, 12345u, d_cycles, d_sink);        // warm-up
    cudaEventRecord(e0);
    probe_kernel<KIND><<<sms, 1024>>>(iters, 12345u, d_cycles, d_sink);
    cudaEventRecord(e1);
    cudaError_t e = cudaEventSynchronize(e1);
    if (e == cudaSuccess) cudaEventElapsedTime(ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return e;
}

}  // namespace

extern "C" int gift_probe_pipe(int device, int kind, uint32_t iters, double* lane_ops_per_clk_per_sm,
                               double* sm_mhz)
{
    if (!lane_ops_per_clk_per_sm || !sm_mhz || iters == 0 || iters > (1u << 20)) return GIFT_E_INVAL;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(device) != cudaSuccess) return GIFT_E_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return GIFT_E_CUDA;
    const int sms = prop.multiProcessorCount;
    unsigned long long* d_cycles = nullptr;
    uint32_t* d_sink = nullptr;
    if (cudaMalloc(&d_cycles, sms * sizeof(unsigned long long)) != cudaSuccess) return GIFT_E_NOMEM;
    if (cudaMalloc(&d_sink, 4) != cudaSuccess) { cudaFree(d_cycles); return GIFT_E_NOMEM; }
    float ms = 0.f;
    cudaError_t e;
    switch (kind) {
    case 0: e = run_probe<0>(sms, iters, d_cycles, d_sink, &ms); break;
    case 1: e = run_probe<1>(sms, iters, d_cycles, d_sink, &ms); break;
    case 2: e = run_probe<2>(sms, iters, d_cycles, d_sink, &ms); break;
    case 3: e = run_probe<3>(sms, iters, d_cycles, d_sink, &ms); break;
    case 4: e = run_probe<4>(sms, iters, d_cycles, d_sink, &ms); break;
    case 5: e = run_probe<5>(sms, iters, d_cycles, d_sink, &ms); break;
    case 6: e = run_probe<6>(sms, iters, d_cycles, d_sink, &ms); break;
    case 7: e = run_probe<7>(sms, iters, d_cycles, d_sink, &ms); break;
    case 8: e = run_probe<8>(sms, iters, d_cycles, d_sink, &ms); break;
    case 9: e = run_probe<9>(sms, iters, d_cycles, d_sink, &ms); break;
    case 10: e = run_probe<10>(sms, iters, d_cycles, d_sink, &ms); break;
    case 11: e = run_probe<11>(sms, iters, d_cycles, d_sink, &ms); break;
    case 12: e = run_probe<12>(sms, iters, d_cycles, d_sink, &ms); break;
    case 13: e = run_probe<13>(sms, iters, d_cycles, d_sink, &ms); break;
    case 14: e = run_probe<14>(sms, iters, d_cycles, d_sink, &ms); break;
    case 15: e = run_probe<15>(sms, iters, d_cycles, d_sink, &ms); break;
    case 16: e = run_probe<16>(sms, iters, d_cycles, d_sink, &ms); break;
    case 17: e = run_probe<17>(sms, iters, d_cycles, d_sink, &ms); break;
    case 18: e = run_probe<18>(sms, iters, d_cycles, d_sink, &ms); break;
    case 19: e = run_probe<19>(sms, iters, d_cycles, d_sink, &ms); break;
    case 20: e = run_probe<20>(sms, iters, d_cycles, d_sink, &ms); break;
    case 21: e = run_probe<21>(sms, iters, d_cycles, d_sink, &ms); break;
    case 22: e = run_probe<22>(sms, iters, d_cycles, d_sink, &ms); break;
    case 23: e = run_probe<23>(sms, iters, d_cycles, d_sink, &ms); break;
    case 24: e = run_probe<24>(sms, iters, d_cycles, d_sink, &ms); break;
    case 25: e = run_probe<25>(sms, iters, d_cycles, d_sink, &ms); break;
    case 26: e = run_probe<26>(sms, iters, d_cycles, d_sink, &ms); break;
    case 27: e = run_probe<27>(sms, iters, d_cycles, d_sink, &ms); break;
    case 28: e = run_probe<28>(sms, iters, d_cycles, d_sink, &ms); break;
    case 29: e = run_probe<29>(sms, iters, d_cycles, d_sink, &ms); break;
    case 30: e = run_probe<30>(sms, iters, d_cycles, d_sink, &ms); break;
    case 31: e = run_probe<31>(sms, iters, d_cycles, d_sink, &ms); break;
    case 32: e = run_probe<32>(sms, iters, d_cycles, d_sink, &ms); break;
    case 33: e = run_probe<33>(sms, iters, d_cycles, d_sink, &ms); break;
    case 34: e = run_probe<34>(sms, iters, d_cycles, d_sink, &ms); break;
    case 35: e = run_probe<35>(sms, iters, d_cycles, d_sink, &ms); break;
    case 36: e = run_probe<36>(sms, iters, d_cycles, d_sink, &ms); break;
    default: cudaFree(d_cycles); cudaFree(d_sink); cudaSetDevice(prev); return GIFT_E_INVAL;
    }
    int rc = GIFT_OK;
    if (e != cudaSuccess) {
        rc = GIFT_E_CUDA;
    } else {
        unsigned long long* h = new unsigned long long[sms];
        cudaMemcpy(h, d_cycles, sms * sizeof(unsigned long long), cudaMemcpyDeviceToHost);
        double mean = 0;
        for (int i = 0; i < sms; i++) mean += (double)h[i];
        mean /= sms;
        delete[] h;
        static const double per_step[37] = {1, 1, 1, 1, 1, 1, 2, 1, 2, 1, 2, 2, 2, 2, 2, 3, 2, 2, 1, 2, 24, 3, 3, 4, 5, 3, 3, 3, 4, 3, 4, 3, 6,
                                            1, 2, 1, 3};
        const double per_pair = per_step[kind];                       // instructions per step
        const double ops = 1024.0 * CHAINS * UNROLL * (double)iters * per_pair;
        *lane_ops_per_clk_per_sm = ops / mean;
        *sm_mhz = mean / (ms * 1e3);
    }
    cudaFree(d_cycles);
    cudaFree(d_sink);
    cudaSetDevice(prev);
    return rc;
}
