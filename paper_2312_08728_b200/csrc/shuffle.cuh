// Per-round shuffle of a buffer (Algorithm 1, "generate random partition of the buffer").
//
// The paper leaves the way the partition is drawn open.  Here round t of chain c under a
// 64-bit seed is a keyed bijection pi on [0, N0): mini-batch m is { pi(j) : m n <= j < (m+1) n }.
// It is stateless, so a thread computes the row it needs and no index array exists in memory.
//
//   round keys  k0..k7 = two blocks of Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) with
//               counter (t, c, 'BMGD', block) and key (seed_lo, seed_hi);
//   bijection   eight rounds of an alternating unbalanced Feistel network on
//               b = max(10, ceil(log2 N0)) bits, round function F(v, k) = hi ^ lo of
//               0xD2511F53 * (v + k); outputs >= N0 are fed back in until one is < N0.
//
// The same bijection, over the whole sample of N rows with the chain word 0xFFFFFFFF and the pass number as
// the round word, is the partition of the sample into buffers that Algorithm 1 draws at the top of each
// pass: buffer k of pass e holds rows pi_e(j), k*N0 <= j < (k+1)*N0.  The host evaluates it while gathering
// rows into the staging buffer, so these functions also compile for the host.
#pragma once
#include <cstdint>

namespace bmgdk {

struct RoundKeys {
    uint32_t k[8];
};

struct FeistelDomain {
    uint32_t N0;
    uint32_t c;      // low-half width in bits
    uint32_t maskA;  // high half
    uint32_t maskC;  // low half
};

__host__ __device__ inline FeistelDomain make_domain(uint32_t N0) {
    uint32_t b = 0;
    while (b < 32 && (1ull << b) < (unsigned long long)N0) ++b;
    if (b < 10) b = 10;
    const uint32_t a = b >> 1, c = b - a;
    FeistelDomain d;
    d.N0 = N0;
    d.c = c;
    d.maskA = (1u << a) - 1u;            // a <= 16
    d.maskC = (c >= 32) ? 0xFFFFFFFFu : ((1u << c) - 1u);
    return d;
}

// high 32 bits of a 32 x 32 -> 64 bit product, on the device and on the host
__host__ __device__ __forceinline__ uint32_t mulhi32(uint32_t a, uint32_t b) {
#ifdef __CUDA_ARCH__
    return __umulhi(a, b);
#else
    return (uint32_t)(((unsigned long long)a * (unsigned long long)b) >> 32);
#endif
}

__host__ __device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                       uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = mulhi32(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = mulhi32(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

__host__ __device__ __forceinline__ RoundKeys round_keys(uint64_t seed, uint32_t chain, uint32_t round) {
    RoundKeys rk;
    const uint32_t klo = (uint32_t)seed, khi = (uint32_t)(seed >> 32);
    philox4x32_10(round, chain, 0x424D4744u, 0u, klo, khi, rk.k);
    philox4x32_10(round, chain, 0x424D4744u, 1u, klo, khi, rk.k + 4);
    return rk;
}

__host__ __device__ __forceinline__ uint32_t feistel_f(uint32_t v, uint32_t k) {
    // one 32 x 32 -> 64 bit multiply gives both halves
    const unsigned long long pr = (unsigned long long)0xD2511F53u * (unsigned long long)(uint32_t)(v + k);
    return (uint32_t)(pr >> 32) ^ (uint32_t)pr;
}

__host__ __device__ __forceinline__ uint32_t perm_index(uint32_t j, const FeistelDomain& d, const RoundKeys& rk) {
    uint32_t x = j;
    do {
        uint32_t L = x >> d.c;
        uint32_t R = x & d.maskC;
#pragma unroll
        for (int r = 0; r < 8; r += 2) {
            L ^= feistel_f(R, rk.k[r]) & d.maskA;
            R ^= feistel_f(L, rk.k[r + 1]) & d.maskC;
        }
        x = (L << d.c) | R;
    } while (x >= d.N0);
    return x;
}

}  // namespace bmgdk
