// CPU oracle for the comparison codec of Appendix B: 1-bit max-norm QSGD, the ternary code that
// snaps coordinate g_i to sign(g_i) with probability |g_i| / ||g||_inf and to 0 otherwise, stored
// in two bits per coordinate ("2d bits can always store d numbers in {0, +-1}").
//
// TEST INFRASTRUCTURE ONLY, like the rest of this directory: plain scalar loops, no code shared
// with the CUDA path, used by the tests alone.
//
// Readings fixed here (Appendix B gives the probabilities, not an encoding or a generator):
//   T1  ||g||_inf is the largest |g_i| over the elements that are not NaN (0 for an empty or
//       all-NaN vector), in fp32.
//   T2  The draw for coordinate c is a 32-bit word r_c; u_c = (r_c >> 9) * 2^-23 is uniform on the
//       2^23 multiples of 2^-23 in [0, 1). The coordinate is kept iff RN(u_c * ||g||_inf) < |g_c|,
//       one rounded fp32 multiply and one comparison: probability |g_c| / ||g||_inf to within
//       2^-23. |g_c| = ||g||_inf is always kept (so a sign vector comes through unchanged, as
//       Appendix B notes), g_c = 0 never, NaN never; if ||g||_inf is Inf nothing is kept.
//   T3  Code of coordinate c: 0 for zero, 1 for +1, 3 for -1 (low bit "kept", high bit
//       "negative"), at bits 2i, 2i+1 of word j for c = 16 j + i; bits beyond d are 0.
//   T4  The draws come from Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers:
//       as easy as 1, 2, 3", SC 2011), the counter-based generator: block b = c / 4 has counter
//       (b mod 2^32, b div 2^32, 0, 0) and key (seed mod 2^32, seed div 2^32); r_c is word c mod 4
//       of that block. Any coordinate's draw can thus be formed without the others.
//   T5  Decoding multiplies the ternary value by a scale (||g||_inf for QSGD's estimate).
//
// Pins (tests/test_oracle_ternary.py): the generator against the known-answer vectors published
// with it; hand-worked keep / drop decisions at the rounding boundary with the draws given as
// inputs; sign vectors unchanged; a single non-zero entry kept alone; 2d bits; the empirical keep
// rate per probability bin and the mean of the decoded value against g over many seeds.

#include <cmath>
#include <cstdint>
#include <cstring>

namespace {

inline float widen_bf16(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return f;
}

inline float grad_at(const void* g, int dtype, int64_t i) {
    if (dtype == 0) return static_cast<const float*>(g)[i];
    return widen_bf16(static_cast<const uint16_t*>(g)[i]);
}

// one round of Philox4x32: two 32 x 32 -> 64 bit products, their halves crossed with the
// counter words and the round key
inline void philox_round(uint32_t c[4], const uint32_t k[2]) {
    const uint64_t p0 = static_cast<uint64_t>(0xD2511F53u) * c[0];
    const uint64_t p1 = static_cast<uint64_t>(0xCD9E8D57u) * c[2];
    const uint32_t hi0 = static_cast<uint32_t>(p0 >> 32), lo0 = static_cast<uint32_t>(p0);
    const uint32_t hi1 = static_cast<uint32_t>(p1 >> 32), lo1 = static_cast<uint32_t>(p1);
    const uint32_t n0 = hi1 ^ c[1] ^ k[0];
    const uint32_t n2 = hi0 ^ c[3] ^ k[1];
    c[0] = n0;
    c[1] = lo1;
    c[2] = n2;
    c[3] = lo0;
}

}  // namespace

extern "C" {

// T4: ten rounds; the key is advanced by the Weyl constants between rounds.
void oracle_philox4x32_10(const uint32_t counter[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c[4] = {counter[0], counter[1], counter[2], counter[3]};
    uint32_t k[2] = {key[0], key[1]};
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k[0] += 0x9E3779B9u;
            k[1] += 0xBB67AE85u;
        }
        philox_round(c, k);
    }
    for (int i = 0; i < 4; ++i) out[i] = c[i];
}

// T4: the draw of every coordinate 0 .. d-1 for a seed.
void oracle_ternary_draws(uint64_t seed, int64_t d, uint32_t* r) {
    const uint32_t key[2] = {static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32)};
    for (int64_t c = 0; c < d; ++c) {
        const uint64_t b = static_cast<uint64_t>(c) / 4;
        const uint32_t counter[4] = {static_cast<uint32_t>(b), static_cast<uint32_t>(b >> 32), 0u, 0u};
        uint32_t out[4];
        oracle_philox4x32_10(counter, key, out);
        r[c] = out[c % 4];
    }
}

// T1
float oracle_absmax(const void* grad, int dtype, int64_t d) {
    float m = 0.0f;
    for (int64_t i = 0; i < d; ++i) {
        const float a = std::fabs(grad_at(grad, dtype, i));
        if (a == a && a > m) m = a;  // NaN is skipped
    }
    return m;
}

int64_t oracle_ternary_words(int64_t d) { return (d + 15) / 16; }

// T2 + T3, with the draws given as an input.
void oracle_ternary_pack(const void* grad, int dtype, int64_t d, float gmax, const uint32_t* r,
                         uint32_t* codes) {
    for (int64_t j = 0; j < oracle_ternary_words(d); ++j) codes[j] = 0u;
    for (int64_t c = 0; c < d; ++c) {
        const float g = grad_at(grad, dtype, c);
        const float u = static_cast<float>(r[c] >> 9) * 1.1920928955078125e-07f;  // exact: 23 bits * 2^-23
        const float t = u * gmax;                                                // one rounded multiply
        const bool kept = t < std::fabs(g);                                      // false for NaN
        uint32_t code = 0u;
        if (kept) code = (g < 0.0f) ? 3u : 1u;
        codes[c / 16] |= code << (2 * (c % 16));
    }
}

// T5
void oracle_ternary_unpack(const uint32_t* codes, int64_t d, float scale, float* out) {
    for (int64_t c = 0; c < d; ++c) {
        const uint32_t code = (codes[c / 16] >> (2 * (c % 16))) & 3u;
        float q = 0.0f;
        if (code & 1u) q = (code & 2u) ? -1.0f : 1.0f;
        out[c] = scale * q;
    }
}

}  // extern "C"
