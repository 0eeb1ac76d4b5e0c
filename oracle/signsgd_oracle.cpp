// CPU oracle for one step of Signum / signSGD with majority vote (Algorithm 1).
//
// TEST INFRASTRUCTURE ONLY. This file is the slow, plain definition that the
// CUDA library is checked against. It shares no code, header, table or helper
// with the CUDA path, and nothing on the product path may call it. It may be
// used only by the tests, by the smoke check and by the benchmark's CPU
// baseline leg.
//
// Style: one coordinate at a time, an integer tally per coordinate, scalar
// loops. No bit-slicing, no vector tricks, no fusion beyond what Algorithm 1
// states. The outer loops run over 32-coordinate blocks only so that two
// threads never write the same packed word when OpenMP is switched on
// (oracle_set_threads); with one thread the order is plain 0..d-1.
//
// Readings of the paper fixed here, once (the paper is silent on each):
//   R1  sign(z) in a 1-bit code: bit = 1 (meaning +1) iff z >= 0 by VALUE.
//       +0.0 and -0.0 both give +1; NaN >= 0 is false, so NaN gives -1;
//       +Inf gives +1, -Inf gives -1.                     (Algorithm 1, "push sign(v_m)")
//   R2  sign(V) for the vote uses the same rule: V >= 0 gives +1, so a tie at
//       even M votes +1.                                  (Algorithm 1, "push sign(V)")
//   R3  Momentum v <- (1-beta) g + beta v is evaluated in fp32 as two rounded
//       multiplies followed by one rounded add, round-to-nearest-even, no fused
//       multiply-add, denormals kept. (1-beta) is formed once in fp32.
//       Build flags: -O2 -ffp-contract=off, no -ffast-math. (Algorithm 1, "update momentum")
//   R4  Update x <- x - eta (sign(V) + lambda x) in fp32, each operation
//       rounded; when lambda == 0 the short form x <- x - (+-eta) is used (it
//       is the same value for finite x and avoids 0*Inf). (Algorithm 1, "update parameters")
//   R5  Packed layout: word j, bit i (bit 0 = least significant) holds
//       coordinate 32 j + i; bits at coordinates >= d are 0 in every output.
//   R6  An inverting adversary complements its sign bits before sending
//       (Section 4.2; proof of Theorem 2), it does not negate its gradient.
//   R7  One momentum buffer per worker (Algorithm 1, "initial momentum v_m <- 0
//       on m-th worker"). bf16 gradients are widened exactly to fp32.
//
// Pins (tests/test_oracle_*.py): brute force over all 2^M sign patterns,
// textbook 3-input majority, numpy little-endian packbits, identical-inputs
// invariant, adversary-survival invariant, geometric-series closed form for
// the momentum, arctan(sigma)/pi and binomial-model vote error rates
// (proof of Theorem 2), hand-computed vectors in tests/golden/.

#include <cstdint>
#include <cstring>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

int g_threads = 1;

inline int64_t words_for(int64_t d) { return (d + 31) / 32; }

// R1: the 1-bit sign.
inline int sign_bit(float z) { return (z >= 0.0f) ? 1 : 0; }

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

// R3: v <- (1-beta) g + beta v, two multiplies then one add, each rounded.
inline float momentum_step(float omb, float g, float beta, float v) {
    float t1 = omb * g;
    float t2 = beta * v;
    return t1 + t2;
}

// R4: x <- x - eta (s + lambda x), s = +-1.
inline float param_step(float x, int bit, float lr, float wd) {
    float s = bit ? 1.0f : -1.0f;
    if (wd == 0.0f) {
        float step = s * lr;  // exact: +-lr
        return x - step;
    }
    float a = wd * x;
    float b = s + a;
    float c = lr * b;
    return x - c;
}

}  // namespace

extern "C" {

// Number of host threads the loops below use (1 = plain serial order).
void oracle_set_threads(int n) { g_threads = n < 1 ? 1 : n; }

int oracle_get_threads(void) { return g_threads; }

int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_num_procs();
#else
    return 1;
#endif
}

// 32x compression: d values become ceil(d/32) words (abstract; Appendix B).
int64_t oracle_packed_words(int64_t d) { return words_for(d); }

// "push sign(g)": one worker's gradient to packed sign bits (R1, R5).
// dtype: 0 = fp32, 1 = bf16 (raw 16-bit patterns).
void oracle_sign_pack(const void* grad, int dtype, int64_t d, uint32_t* out) {
    const int64_t W = words_for(d);
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t j = 0; j < W; ++j) {
        uint32_t w = 0;
        for (int i = 0; i < 32; ++i) {
            int64_t c = 32 * j + i;
            if (c >= d) break;
            if (sign_bit(grad_at(grad, dtype, c))) w |= (1u << i);
        }
        out[j] = w;
    }
}

// Inverse of the packing, to +-1 as int8 (test helper; R5).
void oracle_unpack(const uint32_t* words, int64_t d, int8_t* out) {
    for (int64_t c = 0; c < d; ++c) {
        int bit = (words[c / 32] >> (c % 32)) & 1u;
        out[c] = bit ? 1 : -1;
    }
}

// Server side of Algorithm 1: V = sum_m sign(v_m), output sign(V) (R2), with
// workers named in flip_mask sending the complement of their bits (R6).
// tally_out (optional, may be null) receives V per coordinate.
void oracle_majority_vote(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                          uint32_t* vote, int32_t* tally_out) {
    const int64_t W = words_for(d);
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t j = 0; j < W; ++j) {
        uint32_t w = 0;
        for (int i = 0; i < 32; ++i) {
            int64_t c = 32 * j + i;
            if (c >= d) break;
            int tally = 0;
            for (int m = 0; m < M; ++m) {
                int bit = (packed[m][j] >> i) & 1u;
                if ((flip_mask >> m) & 1u) bit ^= 1;
                tally += bit ? 1 : -1;
            }
            if (tally_out) tally_out[c] = tally;
            if (tally >= 0) w |= (1u << i);
        }
        vote[j] = w;
    }
}

// Worker side of Algorithm 1 with momentum: v <- (1-beta) g + beta v in place,
// then sign(v) packed (R3, R1, R5).
void oracle_signum_update(const void* grad, int dtype, float* momentum, float beta, int64_t d,
                          uint32_t* out) {
    const float omb = 1.0f - beta;
    const int64_t W = words_for(d);
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t j = 0; j < W; ++j) {
        uint32_t w = 0;
        for (int i = 0; i < 32; ++i) {
            int64_t c = 32 * j + i;
            if (c >= d) break;
            float v = momentum_step(omb, grad_at(grad, dtype, c), beta, momentum[c]);
            momentum[c] = v;
            if (sign_bit(v)) w |= (1u << i);
        }
        out[j] = w;
    }
}

// "update parameters": x <- x - eta (sign(V) + lambda x) from the packed vote (R4).
void oracle_apply_vote(float* param, const uint32_t* vote, int64_t d, float lr, float wd) {
    const int64_t W = words_for(d);
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t j = 0; j < W; ++j) {
        for (int i = 0; i < 32; ++i) {
            int64_t c = 32 * j + i;
            if (c >= d) break;
            int bit = (vote[j] >> i) & 1u;
            param[c] = param_step(param[c], bit, lr, wd);
        }
    }
}

// One whole iteration of Algorithm 1 for M simulated workers, coordinate by
// coordinate in the algorithm's order: momentum, sign, (adversary), tally,
// sign of the tally, parameter update. momenta == null means beta = 0 without
// momentum storage (signSGD). vote_out may be null.
void oracle_fused_step(const void* const* grads, int dtype, float* const* momenta, int M,
                       int64_t d, float beta, uint64_t flip_mask, float* param, float lr,
                       float wd, uint32_t* vote_out) {
    const float omb = 1.0f - beta;
    const int64_t W = words_for(d);
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t j = 0; j < W; ++j) {
        uint32_t w = 0;
        for (int i = 0; i < 32; ++i) {
            int64_t c = 32 * j + i;
            if (c >= d) break;
            int tally = 0;
            for (int m = 0; m < M; ++m) {
                float s = grad_at(grads[m], dtype, c);
                if (momenta) {
                    s = momentum_step(omb, s, beta, momenta[m][c]);
                    momenta[m][c] = s;
                }
                int bit = sign_bit(s);
                if ((flip_mask >> m) & 1u) bit ^= 1;
                tally += bit ? 1 : -1;
            }
            int vbit = (tally >= 0) ? 1 : 0;
            if (vbit) w |= (1u << i);
            param[c] = param_step(param[c], vbit, lr, wd);
        }
        if (vote_out) vote_out[j] = w;
    }
}

}  // extern "C"
