// ss_majority_vote and ss_apply_vote kernels: the server's and the workers' halves of
// Algorithm 1 on already packed words (the unfused form a multi-GPU worker would use).
#include <type_traits>

#include "bitslice.cuh"
#include "common.cuh"

namespace ss {

template <int NP>
struct VoteArgs {
    const uint32_t* p[NP];
    uint32_t* out;
    int64_t d;
    uint64_t flip;
    int M;
};

template <int M_CT>
struct VoteShape {
    static constexpr int NP = M_CT > 0 ? M_CT : SS_MAX_WORKERS;
    static constexpr int P = M_CT > 0 ? bit_length(M_CT) : bit_length(SS_MAX_WORKERS);
    static constexpr int LB = M_CT > 0 ? (M_CT < 8 ? M_CT : 8) : 4;
};

// mask of the valid bits of word j (only the last word can be ragged)
__device__ __forceinline__ uint32_t valid_bits(int64_t j, int64_t d) {
    const int64_t W = (d + 31) >> 5;
    const int r = static_cast<int>(d & 31);
    return (j == W - 1 && r != 0) ? ((1u << r) - 1u) : 0xFFFFFFFFu;
}

// one word per thread, 32-bit loads (tail words and the unaligned fallback)
template <int M_CT>
__device__ __forceinline__ void vote_one_word(const VoteArgs<VoteShape<M_CT>::NP>& a, int64_t j) {
    using S = VoteShape<M_CT>;
    constexpr int LB = S::LB;
    const int M = M_CT > 0 ? M_CT : a.M;
    BitCounter<S::P> cnt;
    cnt.clear();
    auto batch = [&](int m0, auto nb_tag) {
        constexpr int NB = decltype(nb_tag)::value;
        uint32_t w[NB];
#pragma unroll
        for (int k = 0; k < NB; ++k) {
            const bool live = (M_CT > 0 || m0 + k < M);
            const int mi = m0 + k < S::NP ? m0 + k : 0;
            w[k] = live ? __ldcs(a.p[mi] + j) : 0u;
        }
#pragma unroll
        for (int k = 0; k < NB; ++k) {
            const bool live = (M_CT > 0 || m0 + k < M);
            if (live && ((a.flip >> (m0 + k)) & 1ull)) w[k] = ~w[k];
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
    const uint32_t T = static_cast<uint32_t>(M + 1) >> 1;
    a.out[j] = cnt.at_least(T) & valid_bits(j, a.d);
}

// four words per thread, 128-bit loads
template <int M_CT>
__global__ void __launch_bounds__(256)
vote_vec_kernel(const __grid_constant__ VoteArgs<VoteShape<M_CT>::NP> a) {
    using S = VoteShape<M_CT>;
    constexpr int LB = S::LB;
    const int M = M_CT > 0 ? M_CT : a.M;
    const int64_t W = (a.d + 31) >> 5;
    const int64_t n_groups = W >> 2;
    const uint32_t T = static_cast<uint32_t>(M + 1) >> 1;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_groups;
         i += stride) {
        BitCounter<S::P> cnt[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) cnt[c].clear();
        auto batch = [&](int m0, auto nb_tag) {
            constexpr int NB = decltype(nb_tag)::value;
            uint4 r[NB];
#pragma unroll
            for (int k = 0; k < NB; ++k) {
                const bool live = (M_CT > 0 || m0 + k < M);
                const int mi = m0 + k < S::NP ? m0 + k : 0;
                r[k] = live ? __ldcs(reinterpret_cast<const uint4*>(a.p[mi]) + i)
                            : make_uint4(0u, 0u, 0u, 0u);
            }
            uint32_t w[4][NB];
#pragma unroll
            for (int k = 0; k < NB; ++k) {
                const bool live = (M_CT > 0 || m0 + k < M);
                const uint32_t f = (live && ((a.flip >> (m0 + k)) & 1ull)) ? 0xFFFFFFFFu : 0u;
                w[0][k] = r[k].x ^ f;
                w[1][k] = r[k].y ^ f;
                w[2][k] = r[k].z ^ f;
                w[3][k] = r[k].w ^ f;
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) cnt[c].template add_words<NB>(w[c]);
        };
        if constexpr (M_CT > 0) {
            constexpr int FULL = M_CT / LB, REM = M_CT % LB;
#pragma unroll
            for (int b = 0; b < FULL; ++b) batch(b * LB, std::integral_constant<int, LB>{});
            if constexpr (REM > 0) batch(FULL * LB, std::integral_constant<int, REM>{});
        } else {
            for (int m0 = 0; m0 < M; m0 += LB) batch(m0, std::integral_constant<int, LB>{});
        }
        uint4 o;
        o.x = cnt[0].at_least(T);
        o.y = cnt[1].at_least(T);
        o.z = cnt[2].at_least(T);
        o.w = cnt[3].at_least(T) & valid_bits(4 * i + 3, a.d);
        __stcs(reinterpret_cast<uint4*>(a.out) + i, o);
    }
    // up to three words that do not fill a group of four
    const int64_t rest = W & 3;
    if (blockIdx.x == 0 && threadIdx.x < rest) vote_one_word<M_CT>(a, (n_groups << 2) + threadIdx.x);
}

template <int M_CT>
__global__ void __launch_bounds__(256)
vote_word_kernel(const __grid_constant__ VoteArgs<VoteShape<M_CT>::NP> a) {
    const int64_t W = (a.d + 31) >> 5;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < W; j += stride)
        vote_one_word<M_CT>(a, j);
}

template <int M_CT, bool VEC>
cudaError_t launch_vote_inst(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                             uint32_t* vote, cudaStream_t st) {
    using S = VoteShape<M_CT>;
    VoteArgs<S::NP> a;
    for (int m = 0; m < S::NP; ++m) a.p[m] = m < M ? packed[m] : nullptr;
    a.out = vote;
    a.d = d;
    a.flip = flip;
    a.M = M;
    const int threads = launch_threads();
    const int64_t W = (d + 31) >> 5;
    int grid = 1;
    cudaError_t err;
    if constexpr (VEC) {
        auto kernel = vote_vec_kernel<M_CT>;
        err = pick_grid(kernel, threads, ((W >> 2) + threads - 1) / threads, &grid);
        if (err != cudaSuccess) return err;
        kernel<<<grid, threads, 0, st>>>(a);
    } else {
        auto kernel = vote_word_kernel<M_CT>;
        err = pick_grid(kernel, threads, (W + threads - 1) / threads, &grid);
        if (err != cudaSuccess) return err;
        kernel<<<grid, threads, 0, st>>>(a);
    }
    return cudaGetLastError();
}

cudaError_t launch_vote(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                        uint32_t* vote, bool vec, cudaStream_t st) {
    if (!vec) return launch_vote_inst<0, false>(packed, M, d, flip, vote, st);
    switch (M) {
        case 1: return launch_vote_inst<1, true>(packed, M, d, flip, vote, st);
        case 3: return launch_vote_inst<3, true>(packed, M, d, flip, vote, st);
        case 7: return launch_vote_inst<7, true>(packed, M, d, flip, vote, st);
        case 15: return launch_vote_inst<15, true>(packed, M, d, flip, vote, st);
        case 16: return launch_vote_inst<16, true>(packed, M, d, flip, vote, st);
        case 31: return launch_vote_inst<31, true>(packed, M, d, flip, vote, st);
        case 63: return launch_vote_inst<63, true>(packed, M, d, flip, vote, st);
        default: return launch_vote_inst<0, true>(packed, M, d, flip, vote, st);
    }
}

// ---- vote + apply in one pass: what a worker does once the other workers' packed signs have
// arrived (Algorithm 1: the server's sum and sign, then "update parameters"). A warp owns a
// tile of 32 packed words = 1024 coordinates: lane l loads word l of every worker (coalesced),
// the bit-sliced counter gives lane l the vote word l, and the 256 quads of x in the tile are
// visited in eight coalesced rounds, each lane fetching the vote word it needs by shuffle. -----

template <int NP>
struct VoteApplyArgs {
    const uint32_t* p[NP];
    uint32_t* out;  // may be null
    float* x;
    int64_t d;
    uint64_t flip;
    float lr, wd;
    const ss_segment* seg;
    int n_seg;
    int M;
};

template <int M_CT, bool VEC, bool SEG>
__global__ void __launch_bounds__(256)
vote_apply_kernel(const __grid_constant__ VoteApplyArgs<VoteShape<M_CT>::NP> a) {
    using S = VoteShape<M_CT>;
    constexpr int LB = S::LB;
    const int M = M_CT > 0 ? M_CT : a.M;
    const int lane = threadIdx.x & 31;
    const int64_t W = (a.d + 31) >> 5;
    const int64_t n_tiles = (W + 31) >> 5;
    const int64_t n_quads = a.d >> 2;  // complete quads of x
    const uint32_t T = static_cast<uint32_t>(M + 1) >> 1;
    const bool has_wd = a.wd != 0.0f;
    const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    for (int64_t t = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; t < n_tiles;
         t += warps) {
        const int64_t j = (t << 5) + lane;
        const bool jv = j < W;
        float4 xq[8];
        if constexpr (VEC) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int64_t Q = (t << 8) + 32 * i + lane;
                if (Q < n_quads) xq[i] = __ldcs(reinterpret_cast<const float4*>(a.x) + Q);
            }
        }
        BitCounter<S::P> cnt;
        cnt.clear();
        auto batch = [&](int m0, auto nb_tag) {
            constexpr int NB = decltype(nb_tag)::value;
            uint32_t w[NB];
#pragma unroll
            for (int k = 0; k < NB; ++k) {
                const bool live = jv && (M_CT > 0 || m0 + k < M);
                const int mi = m0 + k < S::NP ? m0 + k : 0;
                w[k] = live ? __ldcs(a.p[mi] + j) : 0u;
            }
#pragma unroll
            for (int k = 0; k < NB; ++k) {
                const bool live = jv && (M_CT > 0 || m0 + k < M);
                if (live && ((a.flip >> (m0 + k)) & 1ull)) w[k] = ~w[k];
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
        const uint32_t vote = jv ? (cnt.at_least(T) & valid_bits(j, a.d)) : 0u;
        if (a.out != nullptr && jv) __stcs(a.out + j, vote);

        if constexpr (VEC) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t vw = __shfl_sync(0xFFFFFFFFu, vote, 4 * i + (lane >> 3));
                const uint32_t nib = (vw >> (4 * (lane & 7))) & 0xFu;
                const int64_t Q = (t << 8) + 32 * i + lane;
                if (Q < n_quads) {
                    float4 xn;
                    if constexpr (SEG)
                        xn = update_seg4(a.seg, a.n_seg, Q, xq[i], nib);
                    else
                        xn = update_rn4(xq[i], nib, a.lr, a.wd, has_wd);
                    __stcs(reinterpret_cast<float4*>(a.x) + Q, xn);
                } else if (Q == n_quads) {  // up to three coordinates past the last full quad
                    for (int64_t c = Q << 2; c < a.d; ++c) {
                        const uint32_t plus = (nib >> (c & 3)) & 1u;
                        if constexpr (SEG)
                            a.x[c] = update_seg1(a.seg, a.n_seg, c, a.x[c], plus);
                        else
                            a.x[c] = update_rn(a.x[c], plus, a.lr, a.wd, has_wd);
                    }
                }
            }
        } else {
#pragma unroll 8
            for (int i = 0; i < 32; ++i) {
                const uint32_t vw = __shfl_sync(0xFFFFFFFFu, vote, i);
                const int64_t c = (((t << 5) + i) << 5) + lane;
                if (c < a.d) {
                    const uint32_t plus = (vw >> lane) & 1u;
                    if constexpr (SEG)
                        a.x[c] = update_seg1(a.seg, a.n_seg, c, a.x[c], plus);
                    else
                        a.x[c] = update_rn(a.x[c], plus, a.lr, a.wd, has_wd);
                }
            }
        }
    }
}

template <int M_CT, bool VEC, bool SEG>
cudaError_t launch_vote_apply_inst(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                                   float* x, float lr, float wd, const ss_segment* seg, int n_seg,
                                   uint32_t* vote, cudaStream_t st) {
    using S = VoteShape<M_CT>;
    VoteApplyArgs<S::NP> a;
    for (int m = 0; m < S::NP; ++m) a.p[m] = m < M ? packed[m] : nullptr;
    a.out = vote;
    a.x = x;
    a.d = d;
    a.flip = flip;
    a.lr = lr;
    a.wd = wd;
    a.seg = seg;
    a.n_seg = n_seg;
    a.M = M;
    const int threads = launch_threads();
    const int64_t tiles = (((d + 31) >> 5) + 31) >> 5;
    const int64_t per_block = threads / 32;
    int grid = 1;
    auto kernel = vote_apply_kernel<M_CT, VEC, SEG>;
    cudaError_t err = pick_grid(kernel, threads, (tiles + per_block - 1) / per_block, &grid);
    if (err != cudaSuccess) return err;
    kernel<<<grid, threads, 0, st>>>(a);
    return cudaGetLastError();
}

template <bool VEC, bool SEG>
cudaError_t launch_vote_apply_m(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                                float* x, float lr, float wd, const ss_segment* seg, int n_seg,
                                uint32_t* vote, cudaStream_t st) {
#define SS_VA(MV) launch_vote_apply_inst<MV, VEC, SEG>(packed, M, d, flip, x, lr, wd, seg, n_seg, vote, st)
    switch (M) {
        case 1: return SS_VA(1);
        case 3: return SS_VA(3);
        case 7: return SS_VA(7);
        case 15: return SS_VA(15);
        case 16: return SS_VA(16);
        case 31: return SS_VA(31);
        case 63: return SS_VA(63);
        default: return SS_VA(0);
    }
#undef SS_VA
}

cudaError_t launch_vote_apply(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                              float* x, float lr, float wd, bool vec, const ss_segment* seg,
                              int n_seg, uint32_t* vote, cudaStream_t st) {
    if (seg != nullptr)
        return vec ? launch_vote_apply_m<true, true>(packed, M, d, flip, x, lr, wd, seg, n_seg, vote, st)
                   : launch_vote_apply_m<false, true>(packed, M, d, flip, x, lr, wd, seg, n_seg, vote, st);
    return vec ? launch_vote_apply_m<true, false>(packed, M, d, flip, x, lr, wd, seg, n_seg, vote, st)
               : launch_vote_apply_m<false, false>(packed, M, d, flip, x, lr, wd, seg, n_seg, vote, st);
}

// ---- the tally itself: V = sum_m sign(v_m) per coordinate as int8 (a diagnostic: the margin by
// which each vote was won, the quantity Z of Theorem 2's proof). A warp owns 32 words: lane l
// counts word l of every worker bit-sliced, then in eight rounds each lane fetches the count
// planes of the word that holds its four coordinates by shuffle, rebuilds the four counts and
// stores four int8 at once (128 contiguous bytes per warp and round). -----------------------------

template <int NP>
struct TallyArgs {
    const uint32_t* p[NP];
    int8_t* out;
    int64_t d;
    uint64_t flip;
    int M;
    int out_aligned4;
};

template <int M_CT>
__global__ void __launch_bounds__(256)
vote_tally_kernel(const __grid_constant__ TallyArgs<VoteShape<M_CT>::NP> a) {
    using S = VoteShape<M_CT>;
    constexpr int LB = S::LB, P = S::P;
    const int M = M_CT > 0 ? M_CT : a.M;
    const int lane = threadIdx.x & 31;
    const int64_t W = (a.d + 31) >> 5;
    const int64_t n_tiles = (W + 31) >> 5;
    const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    for (int64_t t = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; t < n_tiles;
         t += warps) {
        const int64_t j = (t << 5) + lane;
        const bool jv = j < W;
        BitCounter<P> cnt;
        cnt.clear();
        auto batch = [&](int m0, auto nb_tag) {
            constexpr int NB = decltype(nb_tag)::value;
            uint32_t w[NB];
#pragma unroll
            for (int k = 0; k < NB; ++k) {
                const bool live = jv && (M_CT > 0 || m0 + k < M);
                const int mi = m0 + k < S::NP ? m0 + k : 0;
                w[k] = live ? __ldcs(a.p[mi] + j) : 0u;
            }
#pragma unroll
            for (int k = 0; k < NB; ++k) {
                const bool live = jv && (M_CT > 0 || m0 + k < M);
                if (live && ((a.flip >> (m0 + k)) & 1ull)) w[k] = ~w[k];
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
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int src = 4 * it + (lane >> 3);
            uint32_t pl[P];
#pragma unroll
            for (int q = 0; q < P; ++q) pl[q] = __shfl_sync(0xFFFFFFFFu, cnt.p[q], src);
            const int64_t c0 = (((t << 5) + src) << 5) + 4 * (lane & 7);
            uint32_t four = 0u;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int pos = 4 * (lane & 7) + b;
                int count = 0;
#pragma unroll
                for (int q = 0; q < P; ++q) count |= static_cast<int>((pl[q] >> pos) & 1u) << q;
                const int V = 2 * count - M;
                four |= (static_cast<uint32_t>(V) & 0xFFu) << (8 * b);
            }
            if (c0 + 3 < a.d && a.out_aligned4) {
                *reinterpret_cast<uint32_t*>(a.out + c0) = four;
            } else {
                for (int b = 0; b < 4; ++b)
                    if (c0 + b < a.d) a.out[c0 + b] = static_cast<int8_t>((four >> (8 * b)) & 0xFFu);
            }
        }
    }
}

template <int M_CT>
cudaError_t launch_tally_inst(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                              int8_t* out, cudaStream_t st) {
    using S = VoteShape<M_CT>;
    TallyArgs<S::NP> a;
    for (int m = 0; m < S::NP; ++m) a.p[m] = m < M ? packed[m] : nullptr;
    a.out = out;
    a.d = d;
    a.flip = flip;
    a.M = M;
    a.out_aligned4 = (reinterpret_cast<uintptr_t>(out) & 3) == 0;
    const int threads = launch_threads();
    const int64_t tiles = (((d + 31) >> 5) + 31) >> 5;
    const int64_t per_block = threads / 32;
    int grid = 1;
    auto kernel = vote_tally_kernel<M_CT>;
    cudaError_t err = pick_grid(kernel, threads, (tiles + per_block - 1) / per_block, &grid);
    if (err != cudaSuccess) return err;
    kernel<<<grid, threads, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_tally(const uint32_t* const* packed, int M, int64_t d, uint64_t flip, int8_t* out,
                         cudaStream_t st) {
    switch (M) {
        case 7: return launch_tally_inst<7>(packed, M, d, flip, out, st);
        case 15: return launch_tally_inst<15>(packed, M, d, flip, out, st);
        default: return launch_tally_inst<0>(packed, M, d, flip, out, st);
    }
}

// ---- apply: x <- x - lr (sign(V) + wd x) from packed vote words ------------------------------

struct ApplyArgs {
    float* x;
    const uint32_t* vote;
    int64_t d;
    float lr, wd;
    const ss_segment* seg;  // per-tensor lr / weight decay (SEG kernels only)
    int n_seg;
};

template <bool SEG>
__device__ __forceinline__ void apply_one(const ApplyArgs& a, int64_t c, bool has_wd) {
    const uint32_t w = __ldg(a.vote + (c >> 5));
    const uint32_t plus = (w >> (c & 31)) & 1u;
    if constexpr (SEG)
        a.x[c] = update_seg1(a.seg, a.n_seg, c, a.x[c], plus);
    else
        a.x[c] = update_rn(a.x[c], plus, a.lr, a.wd, has_wd);
}

template <bool SEG>
__global__ void __launch_bounds__(256) apply_vec_kernel(const __grid_constant__ ApplyArgs a) {
    constexpr int U = 4;
    const bool has_wd = a.wd != 0.0f;
    const int64_t n_quads = a.d >> 2;
    const int64_t tile = static_cast<int64_t>(blockDim.x) * U;
    for (int64_t base = static_cast<int64_t>(blockIdx.x) * tile; base < n_quads;
         base += static_cast<int64_t>(gridDim.x) * tile) {
        float4 xq[U];
        uint32_t w[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t q = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            if (q < n_quads) {
                xq[u] = __ldcs(reinterpret_cast<const float4*>(a.x) + q);
                w[u] = __ldg(a.vote + (q >> 3));
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t q = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            if (q < n_quads) {
                const uint32_t nib = (w[u] >> ((q & 7) * 4)) & 0xFu;
                float4 xn;
                if constexpr (SEG)
                    xn = update_seg4(a.seg, a.n_seg, q, xq[u], nib);
                else
                    xn = update_rn4(xq[u], nib, a.lr, a.wd, has_wd);
                __stcs(reinterpret_cast<float4*>(a.x) + q, xn);
            }
        }
    }
    const int64_t rest = a.d & 3;
    if (blockIdx.x == 0 && threadIdx.x < rest) apply_one<SEG>(a, (n_quads << 2) + threadIdx.x, has_wd);
}

template <bool SEG>
__global__ void __launch_bounds__(256) apply_scalar_kernel(const __grid_constant__ ApplyArgs a) {
    const bool has_wd = a.wd != 0.0f;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t c = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; c < a.d; c += stride)
        apply_one<SEG>(a, c, has_wd);
}

cudaError_t launch_apply(float* x, const uint32_t* vote, int64_t d, float lr, float wd, bool vec,
                         const ss_segment* seg, int n_seg, cudaStream_t st) {
    ApplyArgs a{x, vote, d, lr, wd, seg, n_seg};
    const bool segmented = seg != nullptr;
    const int threads = launch_threads();
    int grid = 1;
    cudaError_t err;
    if (vec) {
        const int64_t tile = static_cast<int64_t>(threads) * 4;
        err = pick_grid(apply_vec_kernel<false>, threads, ((d >> 2) + tile - 1) / tile, &grid);
        if (err != cudaSuccess) return err;
        if (segmented)
            apply_vec_kernel<true><<<grid, threads, 0, st>>>(a);
        else
            apply_vec_kernel<false><<<grid, threads, 0, st>>>(a);
    } else {
        err = pick_grid(apply_scalar_kernel<false>, threads, (d + threads - 1) / threads, &grid);
        if (err != cudaSuccess) return err;
        if (segmented)
            apply_scalar_kernel<true><<<grid, threads, 0, st>>>(a);
        else
            apply_scalar_kernel<false><<<grid, threads, 0, st>>>(a);
    }
    return cudaGetLastError();
}

}  // namespace ss
