// The streaming kernel behind ss_sign_pack, ss_signum_update and ss_fused_step: per coordinate,
// Algorithm 1's momentum update, 1-bit sign, majority vote over the M workers and parameter
// update, in one pass over memory.
//
// Vector form: a thread owns U quads (4 consecutive coordinates each). For every worker it
// loads one 128-bit quad of the gradient (64-bit for bf16) and of the momentum, forms a 4-bit
// sign nibble, and feeds the nibbles to a bit-sliced carry-save counter held in registers. The
// vote nibble updates the thread's quad of x; eight neighbouring lanes OR their nibbles into one
// canonical packed word. Loads are issued in batches of LB workers so that several 128-bit
// requests per thread are in flight before the first is consumed.
//
// Ballot form: lane l of a warp owns coordinate 32 j + l of word j; __ballot_sync yields worker
// m's canonical packed word directly and the counter runs on whole words, uniformly across the
// warp. It needs only element alignment, handles the ragged last word, and is the fallback when
// a pointer is not 16-byte aligned.
#pragma once

#include <cuda_bf16.h>
#include <string.h>

#include <type_traits>

#include "bitslice.cuh"
#include "common.cuh"

namespace ss {

template <int NP>
struct StepArgs {
    const void* g[NP];
    float* v[NP];
    uint32_t fnib[NP];  // 0xF for an inverting worker, else 0: XORed into its sign nibble
    float* x;
    uint32_t* words;
    int64_t d;
    uint64_t flip;
    float beta, omb, lr, wd;
    int M;
    const ss_segment* seg;  // per-tensor lr / weight decay (SEG kernels only)
    int n_seg;
};

// Worker quads a thread requests per load batch (twice as many 128-bit loads with momentum).
#ifndef SS_BATCH_MOMENTUM
#define SS_BATCH_MOMENTUM 4
#endif
#ifndef SS_BATCH_PLAIN
#define SS_BATCH_PLAIN 8
#endif

template <int M_CT, bool MOM>
struct StepShape {
    static constexpr int NP = M_CT > 0 ? M_CT : SS_MAX_WORKERS;
    static constexpr int P = M_CT > 0 ? bit_length(M_CT) : bit_length(SS_MAX_WORKERS);
    static constexpr int IN_FLIGHT = MOM ? SS_BATCH_MOMENTUM : SS_BATCH_PLAIN;
    static constexpr int LB = M_CT > 0 ? (M_CT < IN_FLIGHT ? M_CT : IN_FLIGHT) : 4;
    static constexpr int U = (IN_FLIGHT / LB) > 0 ? (IN_FLIGHT / LB) : 1;
};

// One ragged or unaligned word: executed by a full warp, lane = bit position. M_CT = 0 loops
// over the workers at run time (a.M of them, pointers indexed dynamically out of the NP slots).
template <int M_CT, int NP, typename GT, bool MOM, bool APPLY, bool SEG>
__device__ __forceinline__ void step_word_ballot(const StepArgs<NP>& a, int64_t j, int lane) {
    constexpr int P = M_CT > 0 ? bit_length(M_CT) : bit_length(NP);
    constexpr int LB = StepShape<M_CT, MOM>::LB;
    const int M = M_CT > 0 ? M_CT : a.M;
    const int64_t c = 32 * j + lane;
    const bool valid = c < a.d;
    const uint32_t vmask = __ballot_sync(0xFFFFFFFFu, valid);

    BitCounter<P> cnt;
    cnt.clear();
    float xs = 0.0f;
    if (APPLY && valid) xs = a.x[c];

    auto batch = [&](int m0, auto nb_tag) {
        constexpr int NB = decltype(nb_tag)::value;
        float gs[NB], vs[NB];
#pragma unroll
        for (int k = 0; k < NB; ++k) {
            const bool on = valid && (M_CT > 0 || m0 + k < M);
            gs[k] = on ? GT::load1(a.g[m0 + k < NP ? m0 + k : 0], c) : -1.0f;
            if (MOM) vs[k] = on ? ld_rmw(a.v[m0 + k < NP ? m0 + k : 0] + c) : 0.0f;
        }
        uint32_t w[NB];
#pragma unroll
        for (int k = 0; k < NB; ++k) {
            const bool live = (M_CT > 0 || m0 + k < M);
            const bool on = valid && live;
            float s = gs[k];
            if (MOM) {
                s = momentum_rn(a.omb, gs[k], a.beta, vs[k]);
                if (on) __stcs(a.v[m0 + k < NP ? m0 + k : 0] + c, s);
            }
            const uint32_t word = __ballot_sync(0xFFFFFFFFu, on && s >= 0.0f);
            const uint32_t fm = (0u - (a.fnib[m0 + k < NP ? m0 + k : 0] & 1u)) & vmask;
            w[k] = live ? (word ^ fm) : 0u;
        }
        cnt.template add_words<NB>(w);
    };

    if constexpr (M_CT > 0) {
        constexpr int FULL = M_CT / LB, REM = M_CT % LB;
#pragma unroll
        for (int b = 0; b < FULL; ++b) batch(b * LB, std::integral_constant<int, LB>{});
        if constexpr (REM > 0) batch(FULL * LB, std::integral_constant<int, REM>{});
    } else {
        for (int m0 = 0; m0 < M; m0 += LB) batch(m0, std::integral_constant<int, LB>{});
    }

    const uint32_t T = static_cast<uint32_t>(M + 1) >> 1;  // ceil(M/2): a tie votes +1
    const uint32_t vote = cnt.at_least(T) & vmask;
    if (APPLY && valid) {
        if constexpr (SEG)
            a.x[c] = update_seg1(a.seg, a.n_seg, c, xs, (vote >> lane) & 1u);
        else
            a.x[c] = update_rn(xs, (vote >> lane) & 1u, a.lr, a.wd, a.wd != 0.0f);
    }
    if (lane == 0 && a.words != nullptr) a.words[j] = vote;
}


// Packed words from per-thread vote nibbles. Eight neighbouring lanes hold the eight nibbles of
// one word (lane k of the group owns bits 4k..4k+3). Every lane of the warp must call this.
//   U == 8: the 8 lanes x 8 quads of a group form an 8 x 8 matrix of nibbles; a three-stage
//           butterfly transposes it across lanes, after which lane k holds the complete word of
//           quad row k and stores it (3 shuffles per 8 words).
//   else:   an OR tree over the group (3 shuffles per word); the group's first lane stores.
template <int U>
__device__ __forceinline__ void store_words(uint32_t* words, const uint32_t* nib, int64_t base,
                                            int64_t n_quads, int lane) {
    const int k = lane & 7;
    if constexpr (U == 8) {
        uint32_t r = 0u;
#pragma unroll
        for (int u = 0; u < 8; ++u) r |= nib[u] << (4 * u);
        uint32_t o = __shfl_xor_sync(0xFFFFFFFFu, r, 4);
        r = (k & 4) ? ((r & 0xFFFF0000u) | (o >> 16)) : ((r & 0x0000FFFFu) | (o << 16));
        o = __shfl_xor_sync(0xFFFFFFFFu, r, 2);
        r = (k & 2) ? ((r & 0xFF00FF00u) | ((o & 0xFF00FF00u) >> 8))
                    : ((r & 0x00FF00FFu) | ((o & 0x00FF00FFu) << 8));
        o = __shfl_xor_sync(0xFFFFFFFFu, r, 1);
        r = (k & 1) ? ((r & 0xF0F0F0F0u) | ((o & 0xF0F0F0F0u) >> 4))
                    : ((r & 0x0F0F0F0Fu) | ((o & 0x0F0F0F0Fu) << 4));
        const int64_t qk = base + static_cast<int64_t>(k) * blockDim.x + threadIdx.x;
        if (qk < n_quads) words[qk >> 3] = r;
    } else {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            uint32_t w = nib[u] << (4 * k);
            w |= __shfl_xor_sync(0xFFFFFFFFu, w, 1);
            w |= __shfl_xor_sync(0xFFFFFFFFu, w, 2);
            w |= __shfl_xor_sync(0xFFFFFFFFu, w, 4);
            const int64_t qu = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            if (k == 0 && qu < n_quads) words[qu >> 3] = w;
        }
    }
}

// G_PLAIN: policy of the gradient loads (see ld_grad), chosen by the launcher.
template <int M_CT, typename GT, bool MOM, bool APPLY, bool SEG, bool G_PLAIN>
__global__ void __launch_bounds__(256)
step_vec_kernel(const __grid_constant__ StepArgs<StepShape<M_CT, MOM>::NP> a) {
    using S = StepShape<M_CT, MOM>;
    constexpr int LB = S::LB, U = S::U;
    const int M = M_CT > 0 ? M_CT : a.M;
    const int lane = threadIdx.x & 31;
    const int64_t n_quads = (a.d >> 5) << 3;  // quads lying in complete words
    const int64_t tile = static_cast<int64_t>(blockDim.x) * U;
    const uint32_t T = static_cast<uint32_t>(M + 1) >> 1;
    const bool has_wd = a.wd != 0.0f;

    // one tile; WHOLE: the tile lies inside the vector, so no access of it needs a bounds test
    auto do_tile = [&](int64_t base, auto whole_tag) {
        constexpr bool WHOLE = decltype(whole_tag)::value;
        int64_t q[U];
        bool ok[U];
        float4 xq[U];
        BitCounter<S::P> cnt[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            q[u] = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            // uniform over each 8-lane group: n_quads is a multiple of 8
            ok[u] = WHOLE ? true : q[u] < n_quads;
            cnt[u].clear();
            if (APPLY && ok[u]) xq[u] = ld_rmw(reinterpret_cast<const float4*>(a.x) + q[u]);
        }

        auto batch = [&](int m0, auto nb_tag) {
            constexpr int NB = decltype(nb_tag)::value;
            float4 gq[U][NB], vq[U][NB];
#pragma unroll
            for (int u = 0; u < U; ++u) {
#pragma unroll
                for (int k = 0; k < NB; ++k) {
                    const bool on = ok[u] && (M_CT > 0 || m0 + k < M);
                    const int mi = m0 + k < S::NP ? m0 + k : 0;
                    gq[u][k] = on ? GT::template load4<G_PLAIN>(a.g[mi], q[u])
                                  : make_float4(-1.f, -1.f, -1.f, -1.f);
                    if (MOM)
                        vq[u][k] = on ? ld_rmw(reinterpret_cast<const float4*>(a.v[mi]) + q[u])
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                uint32_t nib[NB];
#pragma unroll
                for (int k = 0; k < NB; ++k) {
                    const bool live = (M_CT > 0 || m0 + k < M);
                    const int mi = m0 + k < S::NP ? m0 + k : 0;
                    float4 s = gq[u][k];
                    if (MOM) {
                        s = momentum_rn4(a.omb, gq[u][k], a.beta, vq[u][k]);
                        if (ok[u] && live) __stcs(reinterpret_cast<float4*>(a.v[mi]) + q[u], s);
                    }
                    // an inverting worker's nibble is complemented (mask read from the parameters)
                    nib[k] = live ? (sign_nibble(s) ^ a.fnib[mi]) : 0u;
                }
                cnt[u].template add_words<NB>(nib);
            }
        };

        if constexpr (M_CT > 0) {
            constexpr int FULL = M_CT / LB, REM = M_CT % LB;
#pragma unroll
            for (int b = 0; b < FULL; ++b) batch(b * LB, std::integral_constant<int, LB>{});
            if constexpr (REM > 0) batch(FULL * LB, std::integral_constant<int, REM>{});
        } else {
            for (int m0 = 0; m0 < M; m0 += LB) batch(m0, std::integral_constant<int, LB>{});
        }

        uint32_t vote[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            vote[u] = ok[u] ? (cnt[u].at_least(T) & 0xFu) : 0u;
            if (APPLY && ok[u]) {
                float4 xn;
                if constexpr (SEG)
                    xn = update_seg4(a.seg, a.n_seg, q[u], xq[u], vote[u]);
                else
                    xn = update_rn4(xq[u], vote[u], a.lr, a.wd, has_wd);
                __stcs(reinterpret_cast<float4*>(a.x) + q[u], xn);
            }
        }
        if (a.words != nullptr) store_words<U>(a.words, vote, base, n_quads, lane);
    };

    for (int64_t base = static_cast<int64_t>(blockIdx.x) * tile; base < n_quads;
         base += static_cast<int64_t>(gridDim.x) * tile) {
        // the unguarded body pays where the worker loop is unrolled; the one-worker and
        // run-time-M kernels keep a single (guarded) body, which costs them fewer registers
        if (M_CT >= 3 && base + tile <= n_quads)
            do_tile(base, std::true_type{});
        else
            do_tile(base, std::false_type{});
    }

    // the ragged last word (d not a multiple of 32): one warp, ballot form, run-time worker loop
    if ((a.d & 31) != 0 && blockIdx.x == 0 && threadIdx.x < 32)
        step_word_ballot<(M_CT == 1 ? 1 : 0), S::NP, GT, MOM, APPLY, SEG>(a, a.d >> 5, lane);
}

template <int M_CT, typename GT, bool MOM, bool APPLY, bool SEG>
__global__ void __launch_bounds__(256)
step_ballot_kernel(const __grid_constant__ StepArgs<StepShape<M_CT, MOM>::NP> a) {
    const int lane = threadIdx.x & 31;
    const int64_t W = (a.d + 31) >> 5;
    const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    for (int64_t j = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; j < W;
         j += warps)
        step_word_ballot<M_CT, StepShape<M_CT, MOM>::NP, GT, MOM, APPLY, SEG>(a, j, lane);
}

// Sign packing of one gradient buffer (ss_sign_pack): a pure read stream, so the kernel is kept
// as lean as the arithmetic allows. Quad form: a thread loads U quads (128-bit requests, all
// issued before the first is used), turns each into a sign nibble, and store_words assembles the
// words across the eight lanes that share one. Tiles that lie inside the vector run without
// bounds tests. Measured against a read-only kernel of the same shape it runs at the same rate.
// One block per tile.
// quads (fp32) and octets (bf16) a thread of the packing kernels has in flight: with 8 the fp32
// kernel streams at the rate of a read-only kernel at every size (with 4 it fell 13 % behind)
constexpr int kPackQuads = 8;
constexpr int kPackOctets = 8;
template <typename GT, int U>
__global__ void __launch_bounds__(256)
pack_vec_kernel(const void* __restrict__ g, uint32_t* __restrict__ words, int64_t d) {
    const int lane = threadIdx.x & 31;
    const int64_t n_quads = (d >> 5) << 3;  // quads lying in complete words
    const int64_t tile = static_cast<int64_t>(blockDim.x) * U;
    // one tile; WHOLE: it lies inside the vector and its loads need no bounds test
    auto do_tile = [&](int64_t base, auto whole_tag) {
        constexpr bool WHOLE = decltype(whole_tag)::value;
        float4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t q = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            v[u] = (WHOLE || q < n_quads) ? GT::load4(g, q) : make_float4(-1.f, -1.f, -1.f, -1.f);
        }
        uint32_t nib[U];
#pragma unroll
        for (int u = 0; u < U; ++u) nib[u] = sign_nibble(v[u]);
        store_words<U>(words, nib, base, n_quads, lane);
    };
    for (int64_t base = static_cast<int64_t>(blockIdx.x) * tile; base < n_quads;
         base += static_cast<int64_t>(gridDim.x) * tile) {
        if (base + tile <= n_quads)
            do_tile(base, std::true_type{});
        else
            do_tile(base, std::false_type{});
    }
    // the ragged last word (d not a multiple of 32): one warp, one coordinate per lane
    if ((d & 31) != 0 && blockIdx.x == 0 && threadIdx.x < 32) {
        const int64_t c = ((d >> 5) << 5) + lane;
        const float z = c < d ? GT::load1(g, c) : -1.0f;
        const uint32_t w = __ballot_sync(0xFFFFFFFFu, z >= 0.0f);
        if (lane == 0) words[d >> 5] = w;
    }
}

// Sign bits of the eight bf16 values of a 128-bit load, coordinate i in bit i. One paired
// bf16 comparison per register gives an all-ones or all-zero half per value (by value: +-0 -> 1,
// NaN -> 0, as sign_bit); each register's two halves are masked down to its two bit positions,
// the four registers are OR-ed, and the upper half is folded onto the lower.
__device__ __forceinline__ uint32_t sign_byte_bf16(const uint4& r) {
    const uint32_t raw[4] = {r.x, r.y, r.z, r.w};
    uint32_t t = 0u;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 pair;
        memcpy(&pair, &raw[i], 4);
        const uint32_t ge = __hge2_mask(pair, __float2bfloat162_rn(0.0f));
        t |= ge & ((1u << (2 * i)) | (2u << (2 * i + 16)));
    }
    return (t | (t >> 16)) & 0xFFu;
}

// Packed words from per-thread sign bytes of octets. Four neighbouring lanes hold the four bytes
// of one word (lane k of the group owns bits 8k..8k+7). For every four rows of the tile the 4 x 4
// matrix of bytes held by a group is transposed across its lanes by a two-stage butterfly, after
// which lane k holds the complete word of row 4h + k and stores it (2 shuffles per 4 words).
// Every lane of the warp must call this; U is a multiple of 4.
template <int U>
__device__ __forceinline__ void store_words_oct(uint32_t* words, const uint32_t* byte, int64_t base,
                                                int64_t n_oct, int lane) {
    static_assert(U % 4 == 0, "rows are transposed four at a time");
    const int k = lane & 3;
#pragma unroll
    for (int h = 0; h < U / 4; ++h) {
        uint32_t r = byte[4 * h] | (byte[4 * h + 1] << 8) | (byte[4 * h + 2] << 16) | (byte[4 * h + 3] << 24);
        uint32_t o = __shfl_xor_sync(0xFFFFFFFFu, r, 2);
        r = (k & 2) ? ((r & 0xFFFF0000u) | (o >> 16)) : ((r & 0x0000FFFFu) | (o << 16));
        o = __shfl_xor_sync(0xFFFFFFFFu, r, 1);
        r = (k & 1) ? ((r & 0xFF00FF00u) | ((o & 0xFF00FF00u) >> 8))
                    : ((r & 0x00FF00FFu) | ((o & 0x00FF00FFu) << 8));
        const int64_t ok = base + static_cast<int64_t>(4 * h + k) * blockDim.x + threadIdx.x;
        if (ok < n_oct) words[ok >> 2] = r;
    }
}

// bf16 gradients with a 16-byte aligned pointer: a lane owns U octets (8 consecutive coordinates
// each, one 128-bit request; 64-bit requests top out near half the HBM rate), all loads issued
// before the first is used; four lanes make a word.
template <int U>
__global__ void __launch_bounds__(256)
pack_oct_bf16_kernel(const void* __restrict__ g, uint32_t* __restrict__ words, int64_t d) {
    const int lane = threadIdx.x & 31;
    const int64_t n_oct = (d >> 5) << 2;  // octets lying in complete words
    const int64_t tile = static_cast<int64_t>(blockDim.x) * U;
    // one tile; WHOLE: it lies inside the vector and its loads need no bounds test
    auto do_tile = [&](int64_t base, auto whole_tag) {
        constexpr bool WHOLE = decltype(whole_tag)::value;
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t o = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            v[u] = (WHOLE || o < n_oct) ? ld_stream(reinterpret_cast<const uint4*>(g) + o)
                                        : make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);
        }
        uint32_t byte[U];
#pragma unroll
        for (int u = 0; u < U; ++u) byte[u] = sign_byte_bf16(v[u]);
        store_words_oct<U>(words, byte, base, n_oct, lane);
    };
    for (int64_t base = static_cast<int64_t>(blockIdx.x) * tile; base < n_oct;
         base += static_cast<int64_t>(gridDim.x) * tile) {
        if (base + tile <= n_oct)
            do_tile(base, std::true_type{});
        else
            do_tile(base, std::false_type{});
    }
    if ((d & 31) != 0 && blockIdx.x == 0 && threadIdx.x < 32) {
        const int64_t c = ((d >> 5) << 5) + lane;
        const float z = c < d ? BF16::load1(g, c) : -1.0f;
        const uint32_t w = __ballot_sync(0xFFFFFFFFu, z >= 0.0f);
        if (lane == 0) words[d >> 5] = w;
    }
}

// Ballot form for a gradient pointer that is not 16-byte aligned: lane l owns coordinate
// 32 j + l, __ballot_sync gives word j whole; PACK_WORDS words per warp with all loads issued
// first. Needs only element alignment; the ragged last word falls out of the predication.
constexpr int PACK_WORDS = 8;

template <typename GT>
__global__ void __launch_bounds__(256)
pack_ballot_kernel(const void* __restrict__ g, uint32_t* __restrict__ words, int64_t d) {
    const int lane = threadIdx.x & 31;
    const int64_t W = (d + 31) >> 5;
    const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    for (int64_t j0 = ((static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5) * PACK_WORDS;
         j0 < W; j0 += warps * PACK_WORDS) {
        float s[PACK_WORDS];
#pragma unroll
        for (int k = 0; k < PACK_WORDS; ++k) {
            const int64_t c = ((j0 + k) << 5) + lane;
            s[k] = c < d ? GT::load1(g, c) : -1.0f;  // beyond d: bit 0
        }
        uint32_t mine = 0u;
#pragma unroll
        for (int k = 0; k < PACK_WORDS; ++k) {
            const uint32_t w = __ballot_sync(0xFFFFFFFFu, s[k] >= 0.0f);
            if (lane == k) mine = w;
        }
        if (lane < PACK_WORDS && j0 + lane < W) words[j0 + lane] = mine;
    }
}

template <typename GT>
cudaError_t launch_pack(const StepDesc& s, cudaStream_t st) {
    const int threads = launch_threads();
    int grid = 1;
    cudaError_t err;
    if (GT::kBytes == 2 && (reinterpret_cast<uintptr_t>(s.g[0]) & 15) == 0) {
        constexpr int U = kPackOctets;
        auto kernel = pack_oct_bf16_kernel<U>;
        const int64_t octets = (s.d >> 5) << 2;
        const int64_t tile = static_cast<int64_t>(threads) * U;
        err = pick_grid(kernel, threads, (octets + tile - 1) / tile, &grid);
        if (err != cudaSuccess) return err;
        kernel<<<grid, threads, 0, st>>>(s.g[0], s.words, s.d);
    } else if (s.vec) {
        constexpr int U = kPackQuads;
        auto kernel = pack_vec_kernel<GT, U>;
        const int64_t quads = (s.d >> 5) << 3;
        const int64_t tile = static_cast<int64_t>(threads) * U;
        err = pick_grid(kernel, threads, (quads + tile - 1) / tile, &grid);
        if (err != cudaSuccess) return err;
        kernel<<<grid, threads, 0, st>>>(s.g[0], s.words, s.d);
    } else {
        const int64_t W = (s.d + 31) >> 5;
        const int64_t per_block = static_cast<int64_t>(threads / 32) * PACK_WORDS;
        auto kernel = pack_ballot_kernel<GT>;
        err = pick_grid(kernel, threads, (W + per_block - 1) / per_block, &grid);
        if (err != cudaSuccess) return err;
        kernel<<<grid, threads, 0, st>>>(s.g[0], s.words, s.d);
    }
    return cudaGetLastError();
}

// ss_signum_update with the all-gather of the packed words folded into the producing kernel:
// every word is stored to n destination buffers, which may be other GPUs' memory mapped into
// this process (plain peer stores over NVLink; nothing is read from a peer). The words are 1/96
// of the bytes this kernel moves, so the remote stores ride along with the momentum pass instead
// of a separate collective reading the words back from HBM.
struct PushDests {
    uint32_t* p[SS_MAX_WORKERS];
    int n;
};

template <typename GT, int U>
__global__ void __launch_bounds__(256)
signum_push_kernel(const void* __restrict__ g, float* __restrict__ v, float beta, float omb,
                   int64_t d, const __grid_constant__ PushDests dst) {
    const int lane = threadIdx.x & 31;
    const int k = lane & 7;
    const int64_t n_quads = (d >> 5) << 3;
    const int64_t tile = static_cast<int64_t>(blockDim.x) * U;
    for (int64_t base = static_cast<int64_t>(blockIdx.x) * tile; base < n_quads;
         base += static_cast<int64_t>(gridDim.x) * tile) {
        float4 gq[U], vq[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t q = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            const bool ok = q < n_quads;
            // fp32 gradients plain, bf16 (64-bit requests) evict-first: as measured for ss_signum_update
            gq[u] = ok ? GT::template load4<GT::kBytes == 4>(g, q) : make_float4(-1.f, -1.f, -1.f, -1.f);
            vq[u] = ok ? ld_rmw(reinterpret_cast<const float4*>(v) + q) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t q = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            const bool ok = q < n_quads;
            const float4 s = momentum_rn4(omb, gq[u], beta, vq[u]);
            if (ok) __stcs(reinterpret_cast<float4*>(v) + q, s);
            uint32_t w = (ok ? sign_nibble(s) : 0u) << (4 * k);
            w |= __shfl_xor_sync(0xFFFFFFFFu, w, 1);
            w |= __shfl_xor_sync(0xFFFFFFFFu, w, 2);
            w |= __shfl_xor_sync(0xFFFFFFFFu, w, 4);
            if (k == 0 && ok)
                for (int p = 0; p < dst.n; ++p) dst.p[p][q >> 3] = w;
        }
    }
    if ((d & 31) != 0 && blockIdx.x == 0 && threadIdx.x < 32) {
        const int64_t c = ((d >> 5) << 5) + lane;
        float s = -1.0f;
        if (c < d) {
            s = momentum_rn(omb, GT::load1(g, c), beta, v[c]);
            v[c] = s;
        }
        const uint32_t w = __ballot_sync(0xFFFFFFFFu, c < d && s >= 0.0f);
        if (lane == 0)
            for (int p = 0; p < dst.n; ++p) dst.p[p][d >> 5] = w;
    }
}

// The same for pointers that are only element-aligned: ballot form (lane l owns coordinate
// 32 j + l), PACK_WORDS words per warp, every word stored to all destinations by the lane that
// holds it. Plain stores only, as above.
template <typename GT>
__global__ void __launch_bounds__(256)
signum_push_ballot_kernel(const void* __restrict__ g, float* __restrict__ v, float beta, float omb,
                          int64_t d, const __grid_constant__ PushDests dst) {
    const int lane = threadIdx.x & 31;
    const int64_t W = (d + 31) >> 5;
    const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    for (int64_t j0 = ((static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5) * PACK_WORDS;
         j0 < W; j0 += warps * PACK_WORDS) {
        float gs[PACK_WORDS], vs[PACK_WORDS];
#pragma unroll
        for (int k = 0; k < PACK_WORDS; ++k) {
            const int64_t c = ((j0 + k) << 5) + lane;
            gs[k] = c < d ? GT::load1(g, c) : -1.0f;
            vs[k] = c < d ? ld_rmw(v + c) : 0.0f;
        }
        uint32_t mine = 0u;
#pragma unroll
        for (int k = 0; k < PACK_WORDS; ++k) {
            const int64_t c = ((j0 + k) << 5) + lane;
            const float s = momentum_rn(omb, gs[k], beta, vs[k]);
            if (c < d) __stcs(v + c, s);
            const uint32_t w = __ballot_sync(0xFFFFFFFFu, c < d && s >= 0.0f);
            if (lane == k) mine = w;
        }
        if (lane < PACK_WORDS && j0 + lane < W)
            for (int p = 0; p < dst.n; ++p) dst.p[p][j0 + lane] = mine;
    }
}

template <typename GT>
cudaError_t launch_signum_push(const void* g, float* v, float beta, float omb, int64_t d,
                               uint32_t* const* dests, int n, bool vec, cudaStream_t st) {
    PushDests dst;
    for (int p = 0; p < SS_MAX_WORKERS; ++p) dst.p[p] = p < n ? dests[p] : nullptr;
    dst.n = n;
    const int threads = launch_threads();
    if (!vec) {
        const int64_t W = (d + 31) >> 5;
        const int64_t per_block = static_cast<int64_t>(threads / 32) * PACK_WORDS;
        auto kernel = signum_push_ballot_kernel<GT>;
        int grid = 1;
        cudaError_t err = pick_grid(kernel, threads, (W + per_block - 1) / per_block, &grid);
        if (err != cudaSuccess) return err;
        kernel<<<grid, threads, 0, st>>>(g, v, beta, omb, d, dst);
        return cudaGetLastError();
    }
    constexpr int U = 4;
    auto kernel = signum_push_kernel<GT, U>;
    const int64_t quads = (d >> 5) << 3;
    const int64_t tile = static_cast<int64_t>(threads) * U;
    int grid = 1;
    cudaError_t err = pick_grid(kernel, threads, (quads + tile - 1) / tile, &grid);
    if (err != cudaSuccess) return err;
    kernel<<<grid, threads, 0, st>>>(g, v, beta, omb, d, dst);
    return cudaGetLastError();
}

// Single-worker signSGD (Theorem 1's update, x <- x - eta sign(g); M = 1, no momentum): no vote to
// take, so the step is sign packing and the parameter update in one lean pass: per quad one
// gradient load, one parameter load, the sign nibble, the update, one store, and the packed word
// by an OR tree. `flip` complements the signs (the lone worker is an inverting adversary).
template <typename GT, int U>
__global__ void __launch_bounds__(256)
single_worker_kernel(const void* __restrict__ g, float* __restrict__ x, uint32_t* __restrict__ words,
                     int64_t d, float lr, float wd, uint32_t flip) {
    const int lane = threadIdx.x & 31;
    const int k = lane & 7;
    const int64_t n_quads = (d >> 5) << 3;
    const int64_t tile = static_cast<int64_t>(blockDim.x) * U;
    const bool has_wd = wd != 0.0f;
    const uint32_t fn = flip ? 0xFu : 0u;
    for (int64_t base = static_cast<int64_t>(blockIdx.x) * tile; base < n_quads;
         base += static_cast<int64_t>(gridDim.x) * tile) {
        float4 gq[U], xq[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t q = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            const bool ok = q < n_quads;
            gq[u] = ok ? GT::load4(g, q) : make_float4(-1.f, -1.f, -1.f, -1.f);
            xq[u] = ok ? ld_rmw(reinterpret_cast<const float4*>(x) + q) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t q = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            const bool ok = q < n_quads;
            const uint32_t nib = ok ? (sign_nibble(gq[u]) ^ fn) : 0u;
            if (ok) __stcs(reinterpret_cast<float4*>(x) + q, update_rn4(xq[u], nib, lr, wd, has_wd));
            if (words != nullptr) {
                uint32_t w = nib << (4 * k);
                w |= __shfl_xor_sync(0xFFFFFFFFu, w, 1);
                w |= __shfl_xor_sync(0xFFFFFFFFu, w, 2);
                w |= __shfl_xor_sync(0xFFFFFFFFu, w, 4);
                if (k == 0 && ok) words[q >> 3] = w;
            }
        }
    }
    if ((d & 31) != 0 && blockIdx.x == 0 && threadIdx.x < 32) {
        const int64_t c = ((d >> 5) << 5) + lane;
        const bool valid = c < d;
        const float z = valid ? GT::load1(g, c) : -1.0f;
        const uint32_t vmask = __ballot_sync(0xFFFFFFFFu, valid);
        uint32_t w = __ballot_sync(0xFFFFFFFFu, valid && z >= 0.0f);
        if (flip) w = ~w & vmask;
        if (valid) x[c] = update_rn(x[c], (w >> lane) & 1u, lr, wd, has_wd);
        if (lane == 0 && words != nullptr) words[d >> 5] = w;
    }
}

template <typename GT>
cudaError_t launch_single_worker(const StepDesc& s, cudaStream_t st) {
    const int threads = launch_threads();
    constexpr int U = 4;
    auto kernel = single_worker_kernel<GT, U>;
    const int64_t quads = (s.d >> 5) << 3;
    const int64_t tile = static_cast<int64_t>(threads) * U;
    int grid = 1;
    cudaError_t err = pick_grid(kernel, threads, (quads + tile - 1) / tile, &grid);
    if (err != cudaSuccess) return err;
    kernel<<<grid, threads, 0, st>>>(s.g[0], s.x, s.words, s.d, s.lr, s.wd,
                                     static_cast<uint32_t>(s.flip & 1ull));
    return cudaGetLastError();
}

template <int NP>
void fill_step_args(StepArgs<NP>& a, const StepDesc& s, bool mom) {
    for (int m = 0; m < NP; ++m) {
        a.g[m] = m < s.M ? s.g[m] : nullptr;
        a.v[m] = (mom && m < s.M) ? s.v[m] : nullptr;
        a.fnib[m] = (m < s.M && ((s.flip >> m) & 1ull)) ? 0xFu : 0u;
    }
    a.x = s.x;
    a.words = s.words;
    a.d = s.d;
    a.flip = s.flip;
    a.beta = s.beta;
    a.omb = s.omb;
    a.lr = s.lr;
    a.wd = s.wd;
    a.M = s.M;
    a.seg = s.seg;
    a.n_seg = s.n_seg;
}

template <int M_CT, typename GT, bool MOM, bool APPLY, bool VEC, bool SEG = false>
cudaError_t launch_step_inst(const StepDesc& s, cudaStream_t st) {
    using S = StepShape<M_CT, MOM>;
    StepArgs<S::NP> a;
    fill_step_args(a, s, MOM);
    const int threads = launch_threads();
    int grid = 1;
    cudaError_t err;
    if constexpr (VEC) {
        const int64_t quads = (s.d >> 5) << 3;
        const int64_t tile = static_cast<int64_t>(threads) * S::U;
        err = pick_grid(step_vec_kernel<M_CT, GT, MOM, APPLY, SEG, false>, threads, (quads + tile - 1) / tile, &grid);
        if (err != cudaSuccess) return err;
        // Gradient loads (see ld_grad): plain with momentum; evict-first in the run-time-M kernel
        // without momentum; in the unrolled kernels without momentum plain once the call reads
        // 1.5 GiB of gradients or more (launch option "plain_loads_from_mib"). Measured plain /
        // evict-first, fp32, isolated
        // launches: M = 15: 1.02 at d = 2^24 (1.0 GB), 1.00 at 25.6 M (1.5 GB), 0.97 at 2^26, 0.96
        // at 2^28; M = 7: 1.05 at 2^24 (0.5 GB), 0.97 at 2^26 (1.9 GB) and at 61 M; M = 3: 1.13 at
        // 2^24, 1.02 at 2^26 (0.8 GB), 0.95 at 2^28 (3.2 GB).
        bool plain = MOM;
        if constexpr (!MOM && M_CT > 0)
            plain = static_cast<int64_t>(s.M) * s.d * GT::kBytes >= launch_plain_loads_from_bytes();
        if constexpr (MOM) {
            step_vec_kernel<M_CT, GT, MOM, APPLY, SEG, true><<<grid, threads, 0, st>>>(a);
        } else if constexpr (M_CT == 0) {
            step_vec_kernel<M_CT, GT, MOM, APPLY, SEG, false><<<grid, threads, 0, st>>>(a);
        } else if (plain) {
            step_vec_kernel<M_CT, GT, MOM, APPLY, SEG, true><<<grid, threads, 0, st>>>(a);
        } else {
            step_vec_kernel<M_CT, GT, MOM, APPLY, SEG, false><<<grid, threads, 0, st>>>(a);
        }
    } else {
        auto kernel = step_ballot_kernel<M_CT, GT, MOM, APPLY, SEG>;
        const int64_t W = (s.d + 31) >> 5;
        const int64_t per_block = threads / 32;
        err = pick_grid(kernel, threads, (W + per_block - 1) / per_block, &grid);
        if (err != cudaSuccess) return err;
        kernel<<<grid, threads, 0, st>>>(a);
    }
    return cudaGetLastError();
}

// dispatch on (M, momentum, apply, alignment) for one gradient dtype. The vector form is
// specialised for the worker counts of the paper's experiments and of the sweep (all 2^k - 1,
// plus 16 for the even-M probe); any other M, and every unaligned call, takes the runtime-M form.
// Without momentum, 31 and 63 workers take the runtime-M form as well: fully unrolled, the
// compiler keeps fewer of a thread's loads in flight (40 registers) and the kernel runs 2-5 %
// slower than the run-time loop over batches of four workers on two quads (64 registers).
// bf16 gradients on 16-byte aligned pointers: the octet kernels (step_oct_kernel.cuh)
template <bool SEG>
cudaError_t launch_step_oct(const StepDesc& s, cudaStream_t st);

template <typename GT>
cudaError_t launch_step_dtype(const StepDesc& s, cudaStream_t st) {
    const bool mom = s.v != nullptr;
    const bool apply = s.x != nullptr;
    if constexpr (GT::kBytes == 2) {
        bool oct = s.vec && (apply || mom);  // plain sign packing has an octet kernel of its own
        for (int m = 0; m < s.M; ++m) oct = oct && (reinterpret_cast<uintptr_t>(s.g[m]) & 15) == 0;
        if (oct) return s.seg != nullptr ? launch_step_oct<true>(s, st) : launch_step_oct<false>(s, st);
    }
#define SS_STEP_PICK(MV, AP, VC)                                             \
    (mom ? launch_step_inst<MV, GT, true, AP, VC>(s, st)                     \
         : launch_step_inst<(MV >= 31 ? 0 : MV), GT, false, AP, VC>(s, st))
    if (!apply) {  // per-worker packing: M == 1 by construction
        if (!mom) return launch_pack<GT>(s, st);
        return s.vec ? launch_step_inst<1, GT, true, false, true>(s, st)
                     : launch_step_inst<1, GT, true, false, false>(s, st);
    }
    if (s.seg != nullptr) {  // per-tensor lr / weight decay from the segment table
#define SS_STEP_PICK_SEG(MV, VC)                                                  \
    (mom ? launch_step_inst<MV, GT, true, true, VC, true>(s, st)                  \
         : launch_step_inst<(MV >= 31 ? 0 : MV), GT, false, true, VC, true>(s, st))
        if (!s.vec) return SS_STEP_PICK_SEG(0, false);
        switch (s.M) {
            case 1: return SS_STEP_PICK_SEG(1, true);
            case 3: return SS_STEP_PICK_SEG(3, true);
            case 7: return SS_STEP_PICK_SEG(7, true);
            case 15: return SS_STEP_PICK_SEG(15, true);
            case 16: return SS_STEP_PICK_SEG(16, true);
            case 31: return SS_STEP_PICK_SEG(31, true);
            case 63: return SS_STEP_PICK_SEG(63, true);
            default: return SS_STEP_PICK_SEG(0, true);
        }
#undef SS_STEP_PICK_SEG
    }
    if (!s.vec) return SS_STEP_PICK(0, true, false);
    if (s.M == 1 && !mom) return launch_single_worker<GT>(s, st);
    switch (s.M) {
        case 1: return SS_STEP_PICK(1, true, true);
        case 3: return SS_STEP_PICK(3, true, true);
        case 7: return SS_STEP_PICK(7, true, true);
        case 15: return SS_STEP_PICK(15, true, true);
        case 16: return SS_STEP_PICK(16, true, true);
        case 31: return SS_STEP_PICK(31, true, true);
        case 63: return SS_STEP_PICK(63, true, true);
        default: return SS_STEP_PICK(0, true, true);
    }
#undef SS_STEP_PICK
}

}  // namespace ss
