// Bit-sliced population counting for the majority vote (Algorithm 1: V = sum_m sign(v_m),
// then sign(V)). Each uint32 holds one sign bit for up to 32 coordinates; the per-coordinate
// count of +1 votes is kept as binary digit planes, so the tally V is never materialised.
// A full adder on three words of equal weight is two 3-input boolean ops (LOP3).
#pragma once

#include <stdint.h>

namespace ss {

__host__ __device__ constexpr int bit_length(int n) { return n <= 0 ? 0 : 1 + bit_length(n >> 1); }

// largest K with 2^K - 1 <= n  (n >= 1)
__host__ __device__ constexpr int tree_order(int n) { return bit_length(n + 1) - 1; }

__device__ __forceinline__ void full_add(uint32_t a, uint32_t b, uint32_t c, uint32_t& sum,
                                         uint32_t& carry) {
    sum = a ^ b ^ c;
    carry = (a & b) | (a & c) | (b & c);
}

// Carry-save adder tree: 2^K - 1 words of weight 1 -> K count planes, 2^K - 1 - K full adders.
template <int K>
__device__ __forceinline__ void count_tree(const uint32_t* in, uint32_t* out) {
    if constexpr (K == 1) {
        out[0] = in[0];
    } else {
        constexpr int H = (1 << (K - 1)) - 1;
        uint32_t a[K - 1], b[K - 1];
        count_tree<K - 1>(in, a);
        count_tree<K - 1>(in + H, b);
        uint32_t carry = in[2 * H];
#pragma unroll
        for (int j = 0; j < K - 1; ++j) {
            uint32_t s, c;
            full_add(a[j], b[j], carry, s, c);
            out[j] = s;
            carry = c;
        }
        out[K - 1] = carry;
    }
}

// Count of +1 votes per bit position, as P binary planes (value < 2^P).
template <int P>
struct BitCounter {
    uint32_t p[P];

    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int j = 0; j < P; ++j) p[j] = 0u;
    }

    // count += the K-plane number t (ripple carry; the caller guarantees no overflow)
    template <int K>
    __device__ __forceinline__ void add_planes(const uint32_t* t) {
        uint32_t carry = 0u;
#pragma unroll
        for (int j = 0; j < P; ++j) {
            uint32_t s, c;
            full_add(p[j], j < K ? t[j] : 0u, carry, s, c);
            p[j] = s;
            carry = c;
        }
    }

    // count += N words of weight 1: greedy split into 2^K - 1 sized trees
    template <int N>
    __device__ __forceinline__ void add_words(const uint32_t* w) {
        if constexpr (N > 0) {
            constexpr int K = tree_order(N) < P ? tree_order(N) : P;
            constexpr int USED = (1 << K) - 1;
            uint32_t t[K];
            count_tree<K>(w, t);
            add_planes<K>(t);
            add_words<N - USED>(w + USED);
        }
    }

    // bit = [count >= T], 1 <= T < 2^P: the carry out of count + (2^P - T)
    __device__ __forceinline__ uint32_t at_least(uint32_t T) const {
        const uint32_t addend = (1u << P) - T;
        uint32_t carry = 0u;
#pragma unroll
        for (int j = 0; j < P; ++j) {
            const uint32_t cb = ((addend >> j) & 1u) ? 0xFFFFFFFFu : 0u;
            carry = (p[j] & carry) | (cb & (p[j] | carry));
        }
        return carry;
    }
};

}  // namespace ss
