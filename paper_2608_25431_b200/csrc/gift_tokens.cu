// Token mode (paper sec. 4.5, "Token encryption"): every 64-bit token, extended with a
// 64-bit nonce to one 128-bit block, goes through AES-128 under its owner's key; the
// end-of-sequence token is replaced by a public marker.  One thread per token; batches are
// at most a few hundred thousand tokens, so the kernels are bound by launch latency and by
// the per-thread key fetch, not by any pipe.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "gift_internal.cuh"

using namespace gift;

namespace {

__global__ void tok_encrypt_kernel(const uint32_t* __restrict__ t0g, const KeyHot* __restrict__ hot,
                                   uint32_t max_users, const uint64_t* __restrict__ tokens,
                                   const uint64_t* __restrict__ nonces, const int32_t* __restrict__ owners,
                                   uint32_t n, uint64_t eos, uint4* __restrict__ out, uint32_t* __restrict__ status)
{
    __shared__ uint32_t t0[256];
    for (int i = threadIdx.x; i < 256; i += blockDim.x) t0[i] = t0g[i];
    __syncthreads();
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int32_t o = owners[i];
    const bool ok = o >= 0 && (uint32_t)o < max_users && hot[o].valid != 0;
    status[i] = ok ? 0u : GIFT_ST_NO_KEY;
    if (!ok) { out[i] = make_uint4(0u, 0u, 0u, 0u); return; }
    const uint64_t tok = tokens[i];
    if (tok == eos) { out[i] = make_uint4(~0u, ~0u, ~0u, ~0u); return; }
    const uint64_t nonce = nonces[i];
    uint32_t s[4] = {(uint32_t)tok, (uint32_t)(tok >> 32), (uint32_t)nonce, (uint32_t)(nonce >> 32)};
    PlainTab tb;
    tb.t0 = t0;
    aes128_encrypt(tb, hot[o].rk, s);
    out[i] = make_uint4(s[0], s[1], s[2], s[3]);
}

__global__ void tok_decrypt_kernel(const uint8_t* __restrict__ isboxg, const KeyHot* __restrict__ hot,
                                   uint32_t max_users, const uint4* __restrict__ in,
                                   const int32_t* __restrict__ owners, uint32_t n, uint64_t eos,
                                   uint64_t* __restrict__ tokens, uint64_t* __restrict__ nonces,
                                   uint32_t* __restrict__ status)
{
    __shared__ uint8_t isbox[256];
    for (int i = threadIdx.x; i < 256; i += blockDim.x) isbox[i] = isboxg[i];
    __syncthreads();
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int32_t o = owners[i];
    const bool ok = o >= 0 && (uint32_t)o < max_users && hot[o].valid != 0;
    status[i] = ok ? 0u : GIFT_ST_NO_KEY;
    uint64_t tok = 0, nonce = 0;
    if (ok) {
        const uint4 c = in[i];
        if ((c.x & c.y & c.z & c.w) == ~0u) {
            tok = eos;                                   // the end-of-sequence marker
        } else {
            uint32_t s[4] = {c.x, c.y, c.z, c.w};
            aes128_decrypt(isbox, hot[o].rk, s);
            tok = (uint64_t)s[0] | ((uint64_t)s[1] << 32);
            nonce = (uint64_t)s[2] | ((uint64_t)s[3] << 32);
        }
    }
    tokens[i] = tok;
    if (nonces) nonces[i] = nonce;
}

}  // namespace

extern "C" {

int gift_tok_encrypt(gift_ctx* c, const uint64_t* tokens, const uint64_t* nonces, const int32_t* owners,
                     uint32_t n, uint64_t eos_token, uint8_t* out16, uint32_t* status, void* stream)
{
    if (!c) return GIFT_E_INVAL;
    if (n == 0) return GIFT_OK;
    if (!tokens || !nonces || !owners || !out16 || !status) return GIFT_E_INVAL;
    if ((uintptr_t)out16 & 15) return GIFT_E_ALIGN;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    tok_encrypt_kernel<<<(n + 127) / 128, 128, 0, (cudaStream_t)stream>>>(
        c->d_t0, c->d_hot, c->max_users, tokens, nonces, owners, n, eos_token, reinterpret_cast<uint4*>(out16), status);
    c->launches++;
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}

int gift_tok_decrypt(gift_ctx* c, const uint8_t* in16, const int32_t* owners, uint32_t n, uint64_t eos_token,
                     uint64_t* tokens_out, uint64_t* nonces_out, uint32_t* status, void* stream)
{
    if (!c) return GIFT_E_INVAL;
    if (n == 0) return GIFT_OK;
    if (!in16 || !owners || !tokens_out || !status) return GIFT_E_INVAL;
    if ((uintptr_t)in16 & 15) return GIFT_E_ALIGN;
    DeviceGuard g(c->device);
    if (!g.ok) return GIFT_E_CUDA;
    tok_decrypt_kernel<<<(n + 127) / 128, 128, 0, (cudaStream_t)stream>>>(
        c->d_isbox, c->d_hot, c->max_users, reinterpret_cast<const uint4*>(in16), owners, n, eos_token, tokens_out,
        nonces_out, status);
    c->launches++;
    CU_TRY(cudaGetLastError());
    return GIFT_OK;
}

}  // extern "C"
