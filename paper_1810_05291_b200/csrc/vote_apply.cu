// ss_majority_vote, ss_vote_apply, ss_vote_tally and ss_apply_vote kernels: the server's and the
// workers' halves of Algorithm 1 on already packed words (the form a multi-GPU worker uses).
//
// Worker counts. Kernels are compiled for a capacity CAP of workers; EXACT says that M == CAP
// (loops and the vote threshold fold at compile time). Any other M runs the next larger capacity
// with the loads of the absent workers switched off, so that every M from 1 to 64 gets wide
// loads, a short unrolled worker loop and a counter of bit_length(CAP) planes.
#include <type_traits>

#include "bitslice.cuh"
#include "common.cuh"
#include "exchange.cuh"

namespace ss {

template <int CAP>
struct VoteShape {
    static constexpr int P = bit_length(CAP);     // count planes
    static constexpr int LB = CAP < 8 ? CAP : 8;  // workers per load batch
};

// Calls fn with a compile-time (CAP, EXACT) pair that serves M workers, 1 <= M <= 64.
#define SS_DISPATCH_WORKERS(M, FN)                      \
    do {                                                \
        const int m_ = (M);                             \
        if (m_ == 1) return FN(1, true);                \
        if (m_ == 3) return FN(3, true);                \
        if (m_ < 3) return FN(3, false);                \
        if (m_ == 7) return FN(7, true);                \
        if (m_ < 7) return FN(7, false);                \
        if (m_ == 15) return FN(15, true);              \
        if (m_ < 15) return FN(15, false);              \
        if (m_ == 16) return FN(16, true);              \
        if (m_ == 31) return FN(31, true);              \
        if (m_ < 31) return FN(31, false);              \
        if (m_ == 63) return FN(63, true);              \
        if (m_ < 63) return FN(63, false);              \
        return FN(64, true);                            \
    } while (0)

// mask of the valid bits of word j (only the last word can be ragged)
__device__ __forceinline__ uint32_t valid_bits(int64_t j, int64_t d) {
    const int64_t W = (d + 31) >> 5;
    const int r = static_cast<int>(d & 31);
    return (j == W - 1 && r != 0) ? ((1u << r) - 1u) : 0xFFFFFFFFu;
}

// The tally of Algorithm 1's server line for WPL words per thread: load(m, w) fetches worker m's
// WPL words; workers are taken in batches of LB so that LB loads per thread are in flight; an
// inverting worker's words are complemented; cnt[c] ends as the count of +1 votes of word c.
template <int CAP, bool EXACT, int WPL, typename Load>
__device__ __forceinline__ void tally_words(BitCounter<VoteShape<CAP>::P>* cnt, int M, uint64_t flip,
                                            Load load) {
    constexpr int LB = VoteShape<CAP>::LB;
    auto batch = [&](int m0, auto nb_tag) {
        constexpr int NB = decltype(nb_tag)::value;
        uint32_t r[NB][WPL];
#pragma unroll
        for (int k = 0; k < NB; ++k) {
            if (EXACT || m0 + k < M) {
                load(m0 + k, r[k]);
            } else {
#pragma unroll
                for (int c = 0; c < WPL; ++c) r[k][c] = 0u;
            }
        }
        uint32_t w[WPL][NB];
#pragma unroll
        for (int k = 0; k < NB; ++k) {
            const bool live = EXACT || m0 + k < M;
            const uint32_t f = (live && ((flip >> (m0 + k)) & 1ull)) ? 0xFFFFFFFFu : 0u;
#pragma unroll
            for (int c = 0; c < WPL; ++c) w[c][k] = r[k][c] ^ f;
        }
#pragma unroll
        for (int c = 0; c < WPL; ++c) cnt[c].template add_words<NB>(w[c]);
    };
    constexpr int FULL = CAP / LB, REM = CAP % LB;
#pragma unroll
    for (int b = 0; b < FULL; ++b) batch(b * LB, std::integral_constant<int, LB>{});
    if constexpr (REM > 0) batch(FULL * LB, std::integral_constant<int, REM>{});
}

// ---- vote only -------------------------------------------------------------------------------

template <int CAP>
struct VoteArgs {
    const uint32_t* p[CAP];
    uint32_t* out;
    int64_t d;
    uint64_t flip;
    int M;
};

// one word per thread, 32-bit loads (tail words and the unaligned fallback)
template <int CAP, bool EXACT>
__device__ __forceinline__ void vote_one_word(const VoteArgs<CAP>& a, int64_t j) {
    const int M = EXACT ? CAP : a.M;
    BitCounter<VoteShape<CAP>::P> cnt[1];
    cnt[0].clear();
    tally_words<CAP, EXACT, 1>(cnt, M, a.flip, [&](int m, uint32_t* w) { w[0] = __ldcs(a.p[m] + j); });
    const uint32_t T = static_cast<uint32_t>(M + 1) >> 1;  // ceil(M/2): a tie votes +1
    a.out[j] = cnt[0].at_least(T) & valid_bits(j, a.d);
}

// four words per thread, 128-bit loads
template <int CAP, bool EXACT>
__global__ void __launch_bounds__(256) vote_vec_kernel(const __grid_constant__ VoteArgs<CAP> a) {
    const int M = EXACT ? CAP : a.M;
    const int64_t W = (a.d + 31) >> 5;
    const int64_t n_groups = W >> 2;
    const uint32_t T = static_cast<uint32_t>(M + 1) >> 1;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_groups;
         i += stride) {
        BitCounter<VoteShape<CAP>::P> cnt[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) cnt[c].clear();
        tally_words<CAP, EXACT, 4>(cnt, M, a.flip, [&](int m, uint32_t* w) {
            const uint4 r = __ldcs(reinterpret_cast<const uint4*>(a.p[m]) + i);
            w[0] = r.x, w[1] = r.y, w[2] = r.z, w[3] = r.w;
        });
        uint4 o;
        o.x = cnt[0].at_least(T);
        o.y = cnt[1].at_least(T);
        o.z = cnt[2].at_least(T);
        o.w = cnt[3].at_least(T) & valid_bits(4 * i + 3, a.d);
        __stcs(reinterpret_cast<uint4*>(a.out) + i, o);
    }
    // up to three words that do not fill a group of four
    const int64_t rest = W & 3;
    if (blockIdx.x == 0 && threadIdx.x < rest) vote_one_word<CAP, EXACT>(a, (n_groups << 2) + threadIdx.x);
}

template <int CAP, bool EXACT>
__global__ void __launch_bounds__(256) vote_word_kernel(const __grid_constant__ VoteArgs<CAP> a) {
    const int64_t W = (a.d + 31) >> 5;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < W; j += stride)
        vote_one_word<CAP, EXACT>(a, j);
}

template <int CAP, bool EXACT, bool VEC>
cudaError_t launch_vote_inst(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                             uint32_t* vote, cudaStream_t st) {
    VoteArgs<CAP> a;
    for (int m = 0; m < CAP; ++m) a.p[m] = m < M ? packed[m] : nullptr;
    a.out = vote;
    a.d = d;
    a.flip = flip;
    a.M = M;
    const int threads = launch_threads();
    const int64_t W = (d + 31) >> 5;
    int grid = 1;
    cudaError_t err;
    if constexpr (VEC) {
        auto kernel = vote_vec_kernel<CAP, EXACT>;
        err = pick_grid(kernel, threads, ((W >> 2) + threads - 1) / threads, &grid);
        if (err != cudaSuccess) return err;
        kernel<<<grid, threads, 0, st>>>(a);
    } else {
        auto kernel = vote_word_kernel<CAP, EXACT>;
        err = pick_grid(kernel, threads, (W + threads - 1) / threads, &grid);
        if (err != cudaSuccess) return err;
        kernel<<<grid, threads, 0, st>>>(a);
    }
    return cudaGetLastError();
}

cudaError_t launch_vote(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                        uint32_t* vote, bool vec, cudaStream_t st) {
    // pointers off the 16-byte grid: one word per thread, run-time worker count
    if (!vec) return launch_vote_inst<SS_MAX_WORKERS, false, false>(packed, M, d, flip, vote, st);
#define SS_VOTE(CAPV, EX) launch_vote_inst<CAPV, EX, true>(packed, M, d, flip, vote, st)
    SS_DISPATCH_WORKERS(M, SS_VOTE);
#undef SS_VOTE
}

// ---- vote + apply in one pass: what a worker does once the other workers' packed signs have
// arrived (Algorithm 1: the server's sum and sign, then "update parameters"). -------------------

template <int CAP>
struct VoteApplyArgs {
    const uint32_t* p[CAP];
    uint32_t* out;  // may be null
    float* x;
    int64_t d;
    uint64_t flip;
    float lr, wd;
    const ss_segment* seg;
    int n_seg;
    int M;
    const uint32_t* guard;  // may be null; a non-zero word there makes the whole launch a no-op
};

// true if the launch has been called off: the word at `guard` (written by an earlier kernel of the
// stream, e.g. a wait for the other workers that ran out of time) is not zero
__device__ __forceinline__ bool called_off(const uint32_t* guard) {
    return guard != nullptr && *reinterpret_cast<const volatile uint32_t*>(guard) != 0u;
}

// Pair form (every packed pointer and the vote output 8-byte aligned, x 16-byte aligned). A warp
// owns a tile of 64 packed words = 2048 coordinates: lane l loads words 2l and 2l+1 of every
// worker with one 64-bit request (eight workers' requests in flight per lane), the bit-sliced
// counter leaves it the two vote words, and the 512 quads of x in the tile are visited in 16
// coalesced rounds of 32 quads, the first eight of them requested before the votes are counted
// so that 4 KB of x and 2 KB of packed words per warp are in flight together. In round r lane l
// needs vote word 4r + (l >> 3), which lane 2r + (l >> 4) holds: two shuffles and a select.
// GUARD is the bounds-checked form of the same tile for the one tile that holds the end of the
// vector (words beyond the last, a ragged last word, a last quad of fewer than four coordinates);
// it takes one quad of x at a time so that its checks cost the streaming tiles no registers.
template <int CAP, bool EXACT, bool SEG, bool GUARD>
__device__ __forceinline__ void vote_apply_pair_tile(const VoteApplyArgs<CAP>& a, int64_t t, int lane,
                                                     int M, uint32_t T, bool has_wd) {
    constexpr int XC = GUARD ? 1 : 8;  // quads of x per lane in flight
    const int64_t W = (a.d + 31) >> 5;
    const int64_t n_quads = a.d >> 2;  // complete quads of x
    const int64_t j0 = (t << 6) + 2 * lane;
    const int64_t qbase = (t << 9) + lane;
    float4 xq[XC];
#pragma unroll
    for (int i = 0; i < XC; ++i) {
        const int64_t Q = qbase + 32 * i;
        if (!GUARD || Q < n_quads) xq[i] = __ldcs(reinterpret_cast<const float4*>(a.x) + Q);
    }
    BitCounter<VoteShape<CAP>::P> cnt[2];
    cnt[0].clear();
    cnt[1].clear();
    tally_words<CAP, EXACT, 2>(cnt, M, a.flip, [&](int m, uint32_t* w) {
        if constexpr (GUARD) {
            w[0] = j0 < W ? __ldcs(a.p[m] + j0) : 0u;
            w[1] = j0 + 1 < W ? __ldcs(a.p[m] + j0 + 1) : 0u;
        } else {
            const uint2 r = __ldcs(reinterpret_cast<const uint2*>(a.p[m] + j0));
            w[0] = r.x, w[1] = r.y;
        }
    });
    uint32_t v0 = cnt[0].at_least(T), v1 = cnt[1].at_least(T);
    if constexpr (GUARD) {
        v0 = j0 < W ? (v0 & valid_bits(j0, a.d)) : 0u;
        v1 = j0 + 1 < W ? (v1 & valid_bits(j0 + 1, a.d)) : 0u;
        if (a.out != nullptr) {
            if (j0 < W) __stcs(a.out + j0, v0);
            if (j0 + 1 < W) __stcs(a.out + j0 + 1, v1);
        }
    } else {
        if (a.out != nullptr) __stcs(reinterpret_cast<uint2*>(a.out + j0), make_uint2(v0, v1));
    }
#pragma unroll
    for (int c0 = 0; c0 < 16; c0 += XC) {
        if (c0 > 0) {
#pragma unroll
            for (int i = 0; i < XC; ++i) {
                const int64_t Q = qbase + 32 * (c0 + i);
                if (!GUARD || Q < n_quads) xq[i] = __ldcs(reinterpret_cast<const float4*>(a.x) + Q);
            }
        }
#pragma unroll
        for (int i = 0; i < XC; ++i) {
            const int r = c0 + i;
            const int src = 2 * r + (lane >> 4);
            const uint32_t e = __shfl_sync(0xFFFFFFFFu, v0, src);
            const uint32_t o = __shfl_sync(0xFFFFFFFFu, v1, src);
            const uint32_t vw = ((lane >> 3) & 1) ? o : e;
            const uint32_t nib = (vw >> (4 * (lane & 7))) & 0xFu;
            const int64_t Q = qbase + 32 * r;
            if (!GUARD || Q < n_quads) {
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
    }
}

template <int CAP, bool EXACT, bool SEG>
__global__ void __launch_bounds__(256, 4)
vote_apply_pair_kernel(const __grid_constant__ VoteApplyArgs<CAP> a) {
    if (called_off(a.guard)) return;
    const int M = EXACT ? CAP : a.M;
    const int lane = threadIdx.x & 31;
    const int64_t n_full = a.d >> 11;                          // tiles whose 2048 coordinates all exist
    const int64_t n_tiles = (((a.d + 31) >> 5) + 63) >> 6;     // at most one more
    const uint32_t T = static_cast<uint32_t>(M + 1) >> 1;
    const bool has_wd = a.wd != 0.0f;
    const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    // Tiles are handed out from the end of the vector backwards: the guarded tile, which works
    // through its quads one at a time, then starts with the first block instead of after the last.
    for (int64_t i = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; i < n_tiles;
         i += warps) {
        const int64_t t = n_tiles - 1 - i;
        if (t < n_full)
            vote_apply_pair_tile<CAP, EXACT, SEG, false>(a, t, lane, M, T, has_wd);
        else
            vote_apply_pair_tile<CAP, EXACT, SEG, true>(a, t, lane, M, T, has_wd);
    }
}

// Word form, for packed pointers that are only 4-byte aligned (VEC: x still 16-byte aligned) and
// for an x off the 16-byte grid (!VEC). A warp owns 32 words = 1024 coordinates, lane l loads
// word l of every worker, and x is visited in eight rounds of quads (VEC) or 32 rounds of single
// coordinates, each lane fetching the vote word it needs by shuffle. Run-time worker count.
template <bool VEC, bool SEG>
__global__ void __launch_bounds__(256)
vote_apply_word_kernel(const __grid_constant__ VoteApplyArgs<SS_MAX_WORKERS> a) {
    if (called_off(a.guard)) return;
    constexpr int CAP = SS_MAX_WORKERS;
    const int M = a.M;
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
        BitCounter<VoteShape<CAP>::P> cnt[1];
        cnt[0].clear();
        tally_words<CAP, false, 1>(cnt, M, a.flip,
                                   [&](int m, uint32_t* w) { w[0] = jv ? __ldcs(a.p[m] + j) : 0u; });
        const uint32_t vote = jv ? (cnt[0].at_least(T) & valid_bits(j, a.d)) : 0u;
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

template <int CAP>
void fill_vote_apply_args(VoteApplyArgs<CAP>& a, const uint32_t* const* packed, int M, int64_t d,
                          uint64_t flip, float* x, float lr, float wd, const ss_segment* seg, int n_seg,
                          uint32_t* vote, const uint32_t* guard) {
    a.guard = guard;
    for (int m = 0; m < CAP; ++m) a.p[m] = m < M ? packed[m] : nullptr;
    a.out = vote;
    a.x = x;
    a.d = d;
    a.flip = flip;
    a.lr = lr;
    a.wd = wd;
    a.seg = seg;
    a.n_seg = n_seg;
    a.M = M;
}

template <int CAP, bool EXACT, bool SEG>
cudaError_t launch_vote_apply_pair(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                                   float* x, float lr, float wd, const ss_segment* seg, int n_seg,
                                   uint32_t* vote, const uint32_t* guard, cudaStream_t st) {
    VoteApplyArgs<CAP> a;
    fill_vote_apply_args(a, packed, M, d, flip, x, lr, wd, seg, n_seg, vote, guard);
    const int threads = launch_threads();
    const int64_t tiles = (((d + 31) >> 5) + 63) >> 6;
    const int64_t per_block = threads / 32;
    int grid = 1;
    auto kernel = vote_apply_pair_kernel<CAP, EXACT, SEG>;
    cudaError_t err = pick_grid(kernel, threads, (tiles + per_block - 1) / per_block, &grid);
    if (err != cudaSuccess) return err;
    kernel<<<grid, threads, 0, st>>>(a);
    return cudaGetLastError();
}

template <bool VEC, bool SEG>
cudaError_t launch_vote_apply_word(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                                   float* x, float lr, float wd, const ss_segment* seg, int n_seg,
                                   uint32_t* vote, const uint32_t* guard, cudaStream_t st) {
    VoteApplyArgs<SS_MAX_WORKERS> a;
    fill_vote_apply_args(a, packed, M, d, flip, x, lr, wd, seg, n_seg, vote, guard);
    const int threads = launch_threads();
    const int64_t tiles = (((d + 31) >> 5) + 31) >> 5;
    const int64_t per_block = threads / 32;
    int grid = 1;
    auto kernel = vote_apply_word_kernel<VEC, SEG>;
    cudaError_t err = pick_grid(kernel, threads, (tiles + per_block - 1) / per_block, &grid);
    if (err != cudaSuccess) return err;
    kernel<<<grid, threads, 0, st>>>(a);
    return cudaGetLastError();
}

template <bool SEG>
cudaError_t launch_vote_apply_seg(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                                  float* x, float lr, float wd, bool vec, const ss_segment* seg,
                                  int n_seg, uint32_t* vote, const uint32_t* guard, cudaStream_t st) {
    bool pair = vec && (vote == nullptr || (reinterpret_cast<uintptr_t>(vote) & 7) == 0);
    for (int m = 0; m < M; ++m) pair = pair && (reinterpret_cast<uintptr_t>(packed[m]) & 7) == 0;
    if (!pair)
        return vec ? launch_vote_apply_word<true, SEG>(packed, M, d, flip, x, lr, wd, seg, n_seg, vote, guard, st)
                   : launch_vote_apply_word<false, SEG>(packed, M, d, flip, x, lr, wd, seg, n_seg, vote, guard, st);
#define SS_VA(CAPV, EX) \
    launch_vote_apply_pair<CAPV, EX, SEG>(packed, M, d, flip, x, lr, wd, seg, n_seg, vote, guard, st)
    SS_DISPATCH_WORKERS(M, SS_VA);
#undef SS_VA
}

cudaError_t launch_vote_apply_guarded(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                                      float* x, float lr, float wd, bool vec, const ss_segment* seg,
                                      int n_seg, uint32_t* vote, const uint32_t* guard, cudaStream_t st) {
    return seg != nullptr
               ? launch_vote_apply_seg<true>(packed, M, d, flip, x, lr, wd, vec, seg, n_seg, vote, guard, st)
               : launch_vote_apply_seg<false>(packed, M, d, flip, x, lr, wd, vec, seg, n_seg, vote, guard, st);
}

cudaError_t launch_vote_apply(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                              float* x, float lr, float wd, bool vec, const ss_segment* seg,
                              int n_seg, uint32_t* vote, cudaStream_t st) {
    return launch_vote_apply_guarded(packed, M, d, flip, x, lr, wd, vec, seg, n_seg, vote, nullptr, st);
}

// ---- the tally itself: V = sum_m sign(v_m) per coordinate as int8 (a diagnostic: the margin by
// which each vote was won, the quantity Z of Theorem 2's proof). A warp owns 32 words: lane l
// counts word l of every worker bit-sliced, then in eight rounds each lane fetches the count
// planes of the word that holds its four coordinates by shuffle, rebuilds the four counts and
// stores four int8 at once (128 contiguous bytes per warp and round). -----------------------------

template <int CAP>
struct TallyArgs {
    const uint32_t* p[CAP];
    int8_t* out;
    int64_t d;
    uint64_t flip;
    int M;
    int out_aligned4;
};

template <int CAP, bool EXACT>
__global__ void __launch_bounds__(256) vote_tally_kernel(const __grid_constant__ TallyArgs<CAP> a) {
    constexpr int P = VoteShape<CAP>::P;
    const int M = EXACT ? CAP : a.M;
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
        tally_words<CAP, EXACT, 1>(&cnt, M, a.flip,
                                   [&](int m, uint32_t* w) { w[0] = jv ? __ldcs(a.p[m] + j) : 0u; });
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

template <int CAP, bool EXACT>
cudaError_t launch_tally_inst(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                              int8_t* out, cudaStream_t st) {
    TallyArgs<CAP> a;
    for (int m = 0; m < CAP; ++m) a.p[m] = m < M ? packed[m] : nullptr;
    a.out = out;
    a.d = d;
    a.flip = flip;
    a.M = M;
    a.out_aligned4 = (reinterpret_cast<uintptr_t>(out) & 3) == 0;
    const int threads = launch_threads();
    const int64_t tiles = (((d + 31) >> 5) + 31) >> 5;
    const int64_t per_block = threads / 32;
    int grid = 1;
    auto kernel = vote_tally_kernel<CAP, EXACT>;
    cudaError_t err = pick_grid(kernel, threads, (tiles + per_block - 1) / per_block, &grid);
    if (err != cudaSuccess) return err;
    kernel<<<grid, threads, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_tally(const uint32_t* const* packed, int M, int64_t d, uint64_t flip, int8_t* out,
                         cudaStream_t st) {
    switch (M) {
        case 7: return launch_tally_inst<7, true>(packed, M, d, flip, out, st);
        case 15: return launch_tally_inst<15, true>(packed, M, d, flip, out, st);
        default: return launch_tally_inst<SS_MAX_WORKERS, false>(packed, M, d, flip, out, st);
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

// quads a thread of the apply kernel has in flight (8 measured 6-12 % slower)
constexpr int kApplyQuads = 4;

template <bool SEG>
__global__ void __launch_bounds__(256) apply_vec_kernel(const __grid_constant__ ApplyArgs a) {
    constexpr int U = kApplyQuads;
    const bool has_wd = a.wd != 0.0f;
    const int64_t n_quads = a.d >> 2;
    const int64_t tile = static_cast<int64_t>(blockDim.x) * U;
    // one tile; WHOLE: it lies inside the vector, so no access of it needs a bounds test
    auto do_tile = [&](int64_t base, auto whole_tag) {
        constexpr bool WHOLE = decltype(whole_tag)::value;
        float4 xq[U];
        uint32_t w[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t q = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            if (WHOLE || q < n_quads) {
                xq[u] = __ldcs(reinterpret_cast<const float4*>(a.x) + q);
                w[u] = __ldg(a.vote + (q >> 3));
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t q = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            if (WHOLE || q < n_quads) {
                const uint32_t nib = (w[u] >> ((q & 7) * 4)) & 0xFu;
                float4 xn;
                if constexpr (SEG)
                    xn = update_seg4(a.seg, a.n_seg, q, xq[u], nib);
                else
                    xn = update_rn4(xq[u], nib, a.lr, a.wd, has_wd);
                __stcs(reinterpret_cast<float4*>(a.x) + q, xn);
            }
        }
    };
    for (int64_t base = static_cast<int64_t>(blockIdx.x) * tile; base < n_quads;
         base += static_cast<int64_t>(gridDim.x) * tile) {
        if (base + tile <= n_quads)
            do_tile(base, std::true_type{});
        else
            do_tile(base, std::false_type{});
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
        const int64_t tile = static_cast<int64_t>(threads) * kApplyQuads;
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
