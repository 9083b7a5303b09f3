// Per-round shuffle of a buffer (Algorithm 1, "generate random partition of the buffer").
//
// The paper leaves the way the partition is drawn open.  Here round t of chain c under a
// 64-bit seed is a keyed bijection pi on [0, N0): mini-batch m is { pi(j) : m n <= j < (m+1) n }.
// It is stateless, so a thread computes the row it needs and no index array exists in memory.
//
//   round keys  k0..k7 = two blocks of Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) with
//               counter (t, c, 'BMGD', block) and key (seed_lo, seed_hi);
//   bijection   a value x of [0, a c) is the pair (L, R) = (x div c, x mod c), with
//               a = max(32, ceil(sqrt N0)) and c = max(32, ceil(N0 / a)): the smallest near-square
//               grid that holds N0, so that almost every x is below N0.  Eight rounds alternate
//               L <- (L + G(R, k, a)) mod a  and  R <- (R + G(L, k, c)) mod c, where
//               G(v, k, m) = floor(F m / 2^32) and F = hi ^ lo of 0xD2511F53 * (v + k mod 2^32);
//               outputs >= N0 (a fraction of about 1/sqrt(N0)) are fed back in until one is < N0.
//               Each round is invertible, so pi is a bijection of [0, N0) for every key.
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
    uint32_t a;      // values of the high half
    uint32_t c;      // values of the low half
    uint32_t inv_c;  // ceil(2^32 / c): turns the division by c into a multiplication
};

__host__ __device__ inline FeistelDomain make_domain(uint32_t N0) {
    // floor(sqrt(N0 - 1)) bit by bit; one more is the smallest a with a * a >= N0
    const uint32_t v = N0 > 0 ? N0 - 1u : 0u;
    uint32_t root = 0;
    for (int bit = 15; bit >= 0; --bit) {
        const uint32_t t = root | (1u << bit);
        if ((unsigned long long)t * t <= (unsigned long long)v) root = t;
    }
    uint32_t a = root + 1u;
    if (a < 32u) a = 32u;
    uint32_t c = (uint32_t)(((unsigned long long)N0 + a - 1u) / a);
    if (c < 32u) c = 32u;
    FeistelDomain d;
    d.N0 = N0;
    d.a = a;
    d.c = c;
    d.inv_c = (uint32_t)(0xFFFFFFFFull / c) + 1u;  // c >= 32, so this fits 32 bits
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

// keyed 32-bit hash of one half, scaled into [0, m)
__host__ __device__ __forceinline__ uint32_t feistel_g(uint32_t v, uint32_t k, uint32_t m) {
    // one 32 x 32 -> 64 bit multiply gives both halves
    const unsigned long long pr = (unsigned long long)0xD2511F53u * (unsigned long long)(uint32_t)(v + k);
    return mulhi32((uint32_t)(pr >> 32) ^ (uint32_t)pr, m);
}

// x -> (x div c, x mod c) for x < a c < 2^32.  mulhi(x, ceil(2^32 / c)) is the quotient or one more (the rounding up
// of the reciprocal adds less than one to x / c); one more shows as a remainder that wrapped round.
__host__ __device__ __forceinline__ void feistel_split(uint32_t x, const FeistelDomain& d, uint32_t& L, uint32_t& R) {
    const uint32_t q = mulhi32(x, d.inv_c);
    const uint32_t r = x - q * d.c;
    const bool wrapped = r >= d.c;  // written as selects: a branch here would stand between the chains of several indices
    L = wrapped ? q - 1u : q;
    R = wrapped ? r + d.c : r;
}

// v mod m for v < 2 m, without a branch: v - m wraps round to a huge value exactly when v < m
__host__ __device__ __forceinline__ uint32_t reduce_once(uint32_t v, uint32_t m) {
    const uint32_t w = v - m;
    return w < v ? w : v;
}

// two rounds of the network: both halves are below their moduli before and after
__host__ __device__ __forceinline__ void feistel_round_pair(uint32_t& L, uint32_t& R, uint32_t k_even, uint32_t k_odd,
                                                            const FeistelDomain& d) {
    L = reduce_once(L + feistel_g(R, k_even, d.a), d.a);
    R = reduce_once(R + feistel_g(L, k_odd, d.c), d.c);
}

__host__ __device__ __forceinline__ uint32_t perm_index(uint32_t j, const FeistelDomain& d, const RoundKeys& rk) {
    uint32_t x = j;
    do {
        uint32_t L, R;
        feistel_split(x, d, L, R);
#pragma unroll
        for (int r = 0; r < 8; r += 2) feistel_round_pair(L, R, rk.k[r], rk.k[r + 1], d);
        x = L * d.c + R;
    } while (x >= d.N0);
    return x;
}

}  // namespace bmgdk
