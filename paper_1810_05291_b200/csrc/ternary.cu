// The comparison codec of Appendix B: 1-bit max-norm QSGD. Coordinate g_i becomes sign(g_i) with
// probability |g_i| / ||g||_inf and 0 otherwise, stored in two bits per coordinate. Three kernels:
// the max-norm reduction, the stochastic ternary packing with a counter-based generator evaluated
// in the kernel (no stream of random numbers is read from memory), and the decoder.
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace ss {

int cuda_status_public(cudaError_t e);  // abi.cu

namespace {

// ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC 2011): ten rounds of two 32 x 32 -> 64 bit
// products whose halves are crossed with the counter and the round key; the key advances by the
// two Weyl constants after every round. Block b of the stream for a seed has counter (b, 0, 0)
// split into 32-bit words and key = seed; its four output words are the draws of coordinates
// 4b .. 4b+3, so any quad's draws are formed from its index alone. ------------------------------
struct Draw4 {
    uint32_t r[4];
};

// The ten round keys of a seed (key + round * Weyl constants), formed once on the host and
// handed to the kernel as parameters: the generator then costs four multiplies and two
// three-input XORs per round and no key arithmetic.
struct PhiloxKeys {
    uint32_t k0[10], k1[10];
};

inline PhiloxKeys philox_keys(uint64_t seed) {
    PhiloxKeys k;
    uint32_t a = static_cast<uint32_t>(seed), b = static_cast<uint32_t>(seed >> 32);
    for (int round = 0; round < 10; ++round) {
        k.k0[round] = a;
        k.k1[round] = b;
        a += 0x9E3779B9u;
        b += 0xBB67AE85u;
    }
    return k;
}

__device__ __forceinline__ Draw4 philox4x32_10(uint64_t block, const PhiloxKeys& key) {
    uint32_t c0 = static_cast<uint32_t>(block), c1 = static_cast<uint32_t>(block >> 32), c2 = 0u, c3 = 0u;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ key.k0[round], n2 = hi0 ^ c3 ^ key.k1[round];
        c0 = n0, c1 = lo1, c2 = n2, c3 = lo0;
    }
    return Draw4{{c0, c1, c2, c3}};
}

// Two-bit code of one coordinate: kept iff RN(u * gmax) < |g| with u = (r >> 9) * 2^-23, i.e.
// with probability |g| / gmax to within 2^-23; 1 = +1, 3 = -1, 0 = dropped (also NaN, and every
// coordinate when gmax is 0 or Inf). The 23 bits become the mantissa of a float f in [1, 2), so
// u = f - 1 exactly and needs no integer-to-float conversion, and RN((f - 1) * gmax) is formed by
// one fused multiply-add, f * gmax - gmax: the exact value is the same and it is rounded once.
// (For gmax = Inf the fused form gives NaN where the product gives Inf; neither is < |g|.)
__device__ __forceinline__ uint32_t ternary_code(float g, uint32_t r, float gmax) {
    const float f = __uint_as_float(0x3F800000u | (r >> 9));
    const bool kept = __fmaf_rn(f, gmax, -gmax) < fabsf(g);
    return kept ? (g < 0.0f ? 3u : 1u) : 0u;
}

// ---- ||g||_inf over the elements that are not NaN. Non-negative floats order like their bit
// patterns, so the reduction is an unsigned integer maximum (warp and block reduce, then at most
// one atomic per block into a word that the launch has zeroed). --------------------------------------------------
template <typename GT, bool VEC>
__global__ void __launch_bounds__(256) absmax_kernel(const void* __restrict__ g, int64_t d, unsigned* out) {
    float m = 0.0f;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    const int64_t tid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if constexpr (VEC) {
        constexpr int U = 8;  // quads in flight per thread: a pure read stream wants them all issued first
        const int64_t n_quads = d >> 2;
        const int64_t tile = static_cast<int64_t>(blockDim.x) * U;
        for (int64_t base = static_cast<int64_t>(blockIdx.x) * tile; base < n_quads;
             base += static_cast<int64_t>(gridDim.x) * tile) {
            float4 v[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t q = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
                v[u] = q < n_quads ? GT::load4(g, q) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < U; ++u)
                m = fmaxf(m, fmaxf(fmaxf(fabsf(v[u].x), fabsf(v[u].y)), fmaxf(fabsf(v[u].z), fabsf(v[u].w))));
        }
        if (tid < (d & 3)) m = fmaxf(m, fabsf(GT::load1(g, (n_quads << 2) + tid)));
    } else {
        for (int64_t c = tid; c < d; c += stride) m = fmaxf(m, fabsf(GT::load1(g, c)));
    }
    // fmaxf drops a NaN operand, so m is a non-negative number (or +Inf). Warp maximum, then the
    // block's through shared memory; the block touches the result word only if it would raise it
    // (the word only ever grows, so a stale read can cause a needless atomic, never a missed one).
    __shared__ unsigned warp_max[kMaxBlockThreads / 32];
    unsigned w = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(m));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = w;
    __syncthreads();
    if (threadIdx.x < 32) {
        const int n_warps = (blockDim.x + 31) >> 5;
        w = __reduce_max_sync(0xFFFFFFFFu, threadIdx.x < n_warps ? warp_max[threadIdx.x] : 0u);
        if (threadIdx.x == 0 && w > __ldcg(out)) atomicMax(out, w);
    }
}

// ---- packing: a thread owns a quad (one 128-bit gradient load, one generator block), makes the
// quad's eight code bits, and the four lanes that share a 16-coordinate word assemble it with two
// shuffles. The ragged last word is packed by the first 16 threads of block 0. ------------------
template <typename GT, bool VEC>
__global__ void __launch_bounds__(256)
ternary_pack_kernel(const void* __restrict__ g, int64_t d, const float* __restrict__ gmax_dev,
                    const __grid_constant__ PhiloxKeys seed, uint32_t* __restrict__ codes) {
    const float gmax = __ldg(gmax_dev);
    const int lane = threadIdx.x & 31;
    const int k4 = lane & 3;
    const int64_t n_quads = (d >> 4) << 2;  // quads lying in complete words
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    // The loop runs on the warp's first quad, so that all 32 lanes stay in it for the shuffles;
    // n_quads is a multiple of 4, so the four lanes of a word are inside or outside together.
    for (int64_t b = static_cast<int64_t>(blockIdx.x) * blockDim.x + (threadIdx.x & ~31); b < n_quads;
         b += stride) {
        const int64_t q = b + lane;
        const bool ok = q < n_quads;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ok) {
            if constexpr (VEC) {
                v = GT::load4(g, q);
            } else {
                v.x = GT::load1(g, 4 * q), v.y = GT::load1(g, 4 * q + 1);
                v.z = GT::load1(g, 4 * q + 2), v.w = GT::load1(g, 4 * q + 3);
            }
        }
        const Draw4 dr = philox4x32_10(static_cast<uint64_t>(q), seed);
        const uint32_t byte = ternary_code(v.x, dr.r[0], gmax) | (ternary_code(v.y, dr.r[1], gmax) << 2) |
                              (ternary_code(v.z, dr.r[2], gmax) << 4) | (ternary_code(v.w, dr.r[3], gmax) << 6);
        uint32_t w = byte << (8 * k4);
        w |= __shfl_xor_sync(0xFFFFFFFFu, w, 1);
        w |= __shfl_xor_sync(0xFFFFFFFFu, w, 2);
        if (ok && k4 == 0) codes[q >> 2] = w;
    }
    if ((d & 15) != 0 && blockIdx.x == 0 && threadIdx.x < 32) {
        const int64_t c = ((d >> 4) << 4) + lane;
        uint32_t code = 0u;
        if (lane < 16 && c < d) {
            const Draw4 dr = philox4x32_10(static_cast<uint64_t>(c) >> 2, seed);
            code = ternary_code(GT::load1(g, c), dr.r[c & 3], gmax) << (2 * lane);
        }
        const uint32_t w = __reduce_or_sync(0xFFFFFFFFu, code);
        if (lane == 0) codes[d >> 4] = w;
    }
}

// ---- decoding: out_c = scale * q_c. A warp takes 32 code words (512 coordinates) per pass: one
// coalesced load of a word per lane, then four rounds in which lane l fetches the word that holds
// quad 32 j + l of the pass from the lane that loaded it and stores that quad, so every store
// instruction of the warp covers 512 contiguous bytes. -----------------------------------------------
template <bool VEC>
__global__ void __launch_bounds__(256)
ternary_unpack_kernel(const uint32_t* __restrict__ codes, int64_t d, const float* __restrict__ scale_dev,
                      float* __restrict__ out) {
    const float scale = __ldg(scale_dev);
    const int lane = threadIdx.x & 31;
    const int64_t n_words = (d + 15) >> 4;
    const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    for (int64_t w0 = ((static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5) << 5; w0 < n_words;
         w0 += warps << 5) {
        const uint32_t mine = w0 + lane < n_words ? __ldg(codes + w0 + lane) : 0u;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t word = __shfl_sync(0xFFFFFFFFu, mine, 8 * j + (lane >> 2));
            const int64_t q = (w0 << 2) + 32 * j + lane;
            const uint32_t byte = (word >> (8 * (lane & 3))) & 0xFFu;
            float f[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t code = (byte >> (2 * i)) & 3u;
                const float t = (code & 1u) ? ((code & 2u) ? -1.0f : 1.0f) : 0.0f;
                f[i] = __fmul_rn(scale, t);
            }
            if (VEC && 4 * q + 3 < d) {
                __stcs(reinterpret_cast<float4*>(out) + q, make_float4(f[0], f[1], f[2], f[3]));
            } else {
                for (int i = 0; i < 4; ++i)
                    if (4 * q + i < d) out[4 * q + i] = f[i];
            }
        }
    }
}

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

inline bool ranges_overlap(const void* p, size_t n, const void* q, size_t m) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(p), b = reinterpret_cast<uintptr_t>(q);
    return n != 0 && m != 0 && a < b + m && b < a + n;
}

inline cudaError_t stream_grid(int threads, int64_t items, int per_sm, int* grid) {
    // grid-stride kernels: enough blocks to cover the items, at most per_sm blocks per SM
    cudaError_t err = cudaSuccess;
    const int sms = device_sm_count(&err);
    if (err != cudaSuccess) return err;
    int64_t blocks = (items + threads - 1) / threads;
    const int64_t cap = static_cast<int64_t>(sms) * per_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    *grid = static_cast<int>(blocks);
    return cudaSuccess;
}

}  // namespace
}  // namespace ss

using namespace ss;

extern "C" {
#pragma GCC visibility push(default)

int64_t ss_ternary_words(int64_t d) { return d < 0 ? -1 : (d + 15) / 16; }

int ss_absmax(const void* grad, ss_dtype dt, int64_t d, float* absmax_dev, void* cuda_stream) {
    if ((dt != SS_F32 && dt != SS_BF16) || d < 0 || d > SS_MAX_COORDS || absmax_dev == nullptr)
        return SS_ERR_INVALID_ARG;
    if (d > 0 && grad == nullptr) return SS_ERR_INVALID_ARG;
    const size_t eb = dt == SS_F32 ? 4 : 2;
    if (!aligned_to(absmax_dev, 4) || (d > 0 && !aligned_to(grad, eb))) return SS_ERR_MISALIGNED;
    if (d > 0 && ranges_overlap(grad, static_cast<size_t>(d) * eb, absmax_dev, 4)) return SS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaMemsetAsync(absmax_dev, 0, 4, st);  // the maximum of nothing is 0
    if (e != cudaSuccess) return cuda_status_public(e);
    if (d == 0) return SS_OK;
    const bool vec = aligned_to(grad, eb * 4);
    const int threads = launch_threads();
    int grid = 1;
    unsigned* out = reinterpret_cast<unsigned*>(absmax_dev);
    // the quad form takes tiles of 8 quads per thread (plus a block's worth for the ragged end)
    const int64_t items = vec ? (d >> 2) / 8 + threads : d;
#define SS_ABSMAX(GT, VEC)                                                        \
    do {                                                                          \
        e = VEC ? pick_grid(absmax_kernel<GT, VEC>, threads, (items + threads - 1) / threads, &grid) \
                : stream_grid(threads, items, 16, &grid);                         \
        if (e != cudaSuccess) return cuda_status_public(e);                       \
        absmax_kernel<GT, VEC><<<grid, threads, 0, st>>>(grad, d, out);           \
    } while (0)
    if (dt == SS_F32) {
        if (vec) SS_ABSMAX(F32, true); else SS_ABSMAX(F32, false);
    } else {
        if (vec) SS_ABSMAX(BF16, true); else SS_ABSMAX(BF16, false);
    }
#undef SS_ABSMAX
    return cuda_status_public(cudaGetLastError());
}

int ss_ternary_pack(const void* grad, ss_dtype dt, int64_t d, const float* absmax_dev, uint64_t seed,
                    uint32_t* out_codes, void* cuda_stream) {
    if ((dt != SS_F32 && dt != SS_BF16) || d < 0 || d > SS_MAX_COORDS) return SS_ERR_INVALID_ARG;
    if (d == 0) return SS_OK;
    if (grad == nullptr || absmax_dev == nullptr || out_codes == nullptr) return SS_ERR_INVALID_ARG;
    const size_t eb = dt == SS_F32 ? 4 : 2;
    if (!aligned_to(grad, eb) || !aligned_to(absmax_dev, 4) || !aligned_to(out_codes, 4)) return SS_ERR_MISALIGNED;
    const size_t gbytes = static_cast<size_t>(d) * eb, cbytes = static_cast<size_t>((d + 15) / 16) * 4;
    if (ranges_overlap(out_codes, cbytes, grad, gbytes) || ranges_overlap(out_codes, cbytes, absmax_dev, 4))
        return SS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const bool vec = aligned_to(grad, eb * 4);
    const int threads = launch_threads();
    int grid = 1;
    cudaError_t e;
    const int64_t quads = ((d >> 4) << 2);
    const PhiloxKeys keys = philox_keys(seed);
#define SS_TPACK(GT, VEC)                                                                  \
    do {                                                                                   \
        e = pick_grid(ternary_pack_kernel<GT, VEC>, threads, (quads + threads - 1) / threads, &grid); \
        if (e != cudaSuccess) return cuda_status_public(e);                                \
        ternary_pack_kernel<GT, VEC><<<grid, threads, 0, st>>>(grad, d, absmax_dev, keys, out_codes); \
    } while (0)
    if (dt == SS_F32) {
        if (vec) SS_TPACK(F32, true); else SS_TPACK(F32, false);
    } else {
        if (vec) SS_TPACK(BF16, true); else SS_TPACK(BF16, false);
    }
#undef SS_TPACK
    return cuda_status_public(cudaGetLastError());
}

int ss_ternary_unpack(const uint32_t* codes, int64_t d, const float* scale_dev, float* out, void* cuda_stream) {
    if (d < 0 || d > SS_MAX_COORDS) return SS_ERR_INVALID_ARG;
    if (d == 0) return SS_OK;
    if (codes == nullptr || scale_dev == nullptr || out == nullptr) return SS_ERR_INVALID_ARG;
    if (!aligned_to(codes, 4) || !aligned_to(scale_dev, 4) || !aligned_to(out, 4)) return SS_ERR_MISALIGNED;
    const size_t obytes = static_cast<size_t>(d) * 4, cbytes = static_cast<size_t>((d + 15) / 16) * 4;
    if (ranges_overlap(out, obytes, codes, cbytes) || ranges_overlap(out, obytes, scale_dev, 4))
        return SS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int threads = launch_threads();
    int grid = 1;
    const int64_t words = (d + 15) >> 4;  // one word per lane and pass
    cudaError_t e = pick_grid(ternary_unpack_kernel<true>, threads, (words + threads - 1) / threads, &grid);
    if (e != cudaSuccess) return cuda_status_public(e);
    if (aligned_to(out, 16))
        ternary_unpack_kernel<true><<<grid, threads, 0, st>>>(codes, d, scale_dev, out);
    else
        ternary_unpack_kernel<false><<<grid, threads, 0, st>>>(codes, d, scale_dev, out);
    return cuda_status_public(cudaGetLastError());
}

#pragma GCC visibility pop
}  // extern "C"
