// Octet form of the streaming step kernel for bf16 gradients whose pointers are 16-byte aligned.
//
// In the quad form a thread's bf16 gradient request is 64 bits wide, and requests of that width
// reach only about half the HBM rate that 128-bit requests do. Here a thread owns U octets (8
// consecutive coordinates each): per worker one 128-bit load brings the eight bf16 gradients and
// two 128-bit loads the eight fp32 momenta, so every request of the kernel is 128 bits wide. The
// eight sign bits of a worker fill one byte of the bit-sliced counter's planes; the vote byte
// updates the thread's two quads of x, and the four lanes that share a packed word assemble it
// with two shuffles. Arithmetic, sign rule and results are those of the quad form.
#pragma once

#include "step_kernel.cuh"

namespace ss {

// the eight bf16 values of a 128-bit load, widened exactly to fp32: coordinates 0-3 and 4-7
__device__ __forceinline__ void widen_octet(const uint4& r, float4& lo, float4& hi) {
    lo.x = __uint_as_float(r.x << 16);
    lo.y = __uint_as_float(r.x & 0xFFFF0000u);
    lo.z = __uint_as_float(r.y << 16);
    lo.w = __uint_as_float(r.y & 0xFFFF0000u);
    hi.x = __uint_as_float(r.z << 16);
    hi.y = __uint_as_float(r.z & 0xFFFF0000u);
    hi.z = __uint_as_float(r.w << 16);
    hi.w = __uint_as_float(r.w & 0xFFFF0000u);
}

// Worker octets a thread requests per load batch: with momentum a worker costs three 128-bit
// requests (48 bytes), without it one.
template <int M_CT, bool MOM>
struct OctShape {
    static constexpr int NP = M_CT > 0 ? M_CT : SS_MAX_WORKERS;
    static constexpr int P = M_CT > 0 ? bit_length(M_CT) : bit_length(SS_MAX_WORKERS);
    static constexpr int IN_FLIGHT = MOM ? 4 : 8;
    static constexpr int LB = M_CT > 0 ? (M_CT < IN_FLIGHT ? M_CT : IN_FLIGHT) : 4;
    static constexpr int U = (IN_FLIGHT / LB) > 0 ? (IN_FLIGHT / LB) : 1;
};

template <int M_CT, bool MOM, bool APPLY, bool SEG>
__global__ void __launch_bounds__(256)
step_oct_bf16_kernel(const __grid_constant__ StepArgs<OctShape<M_CT, MOM>::NP> a) {
    using S = OctShape<M_CT, MOM>;
    constexpr int LB = S::LB, U = S::U;
    // loads: plain in the fused step, evict-first throughout in the one-worker momentum update (see ld_grad)
    constexpr bool G_PLAIN = APPLY;
    const int M = M_CT > 0 ? M_CT : a.M;
    const int lane = threadIdx.x & 31;
    const int k4 = lane & 3;
    const int64_t n_oct = (a.d >> 5) << 2;  // octets lying in complete words
    const int64_t tile = static_cast<int64_t>(blockDim.x) * U;
    const uint32_t T = static_cast<uint32_t>(M + 1) >> 1;
    const bool has_wd = a.wd != 0.0f;

    for (int64_t base = static_cast<int64_t>(blockIdx.x) * tile; base < n_oct;
         base += static_cast<int64_t>(gridDim.x) * tile) {
        int64_t o[U];
        bool ok[U];
        float4 xlo[U], xhi[U];
        BitCounter<S::P> cnt[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            o[u] = base + static_cast<int64_t>(u) * blockDim.x + threadIdx.x;
            ok[u] = o[u] < n_oct;  // uniform over each 4-lane group: n_oct is a multiple of 4
            cnt[u].clear();
            if (APPLY && ok[u]) {
                xlo[u] = ld_rmw(reinterpret_cast<const float4*>(a.x) + 2 * o[u]);
                xhi[u] = ld_rmw(reinterpret_cast<const float4*>(a.x) + 2 * o[u] + 1);
            }
        }

        auto batch = [&](int m0, auto nb_tag) {
            constexpr int NB = decltype(nb_tag)::value;
            uint4 gq[U][NB];
            float4 vlo[U][NB], vhi[U][NB];
#pragma unroll
            for (int u = 0; u < U; ++u) {
#pragma unroll
                for (int k = 0; k < NB; ++k) {
                    const bool on = ok[u] && (M_CT > 0 || m0 + k < M);
                    const int mi = m0 + k < S::NP ? m0 + k : 0;
                    gq[u][k] = on ? ld_grad<G_PLAIN>(reinterpret_cast<const uint4*>(a.g[mi]) + o[u])
                                  : make_uint4(0x80008000u, 0x80008000u, 0x80008000u, 0x80008000u);
                    if (MOM) {
                        const float4* vp = reinterpret_cast<const float4*>(a.v[mi]) + 2 * o[u];
                        vlo[u][k] = on ? ld_rmw_as<G_PLAIN>(vp) : make_float4(0.f, 0.f, 0.f, 0.f);
                        vhi[u][k] = on ? ld_rmw_as<G_PLAIN>(vp + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                uint32_t bits[NB];
#pragma unroll
                for (int k = 0; k < NB; ++k) {
                    const bool live = (M_CT > 0 || m0 + k < M);
                    const int mi = m0 + k < S::NP ? m0 + k : 0;
                    float4 slo, shi;
                    widen_octet(gq[u][k], slo, shi);
                    if (MOM) {
                        slo = momentum_rn4(a.omb, slo, a.beta, vlo[u][k]);
                        shi = momentum_rn4(a.omb, shi, a.beta, vhi[u][k]);
                        if (ok[u] && live) {
                            float4* vp = reinterpret_cast<float4*>(a.v[mi]) + 2 * o[u];
                            __stcs(vp, slo);
                            __stcs(vp + 1, shi);
                        }
                    }
                    // an inverting worker's byte is complemented (mask from the parameters)
                    const uint32_t fbyte = (0u - (a.fnib[mi] & 1u)) & 0xFFu;
                    bits[k] = live ? ((sign_nibble(slo) | (sign_nibble(shi) << 4)) ^ fbyte) : 0u;
                }
                cnt[u].template add_words<NB>(bits);
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

#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t vote = ok[u] ? (cnt[u].at_least(T) & 0xFFu) : 0u;
            if (APPLY && ok[u]) {
                float4 nlo, nhi;
                if constexpr (SEG) {
                    nlo = update_seg4(a.seg, a.n_seg, 2 * o[u], xlo[u], vote & 0xFu);
                    nhi = update_seg4(a.seg, a.n_seg, 2 * o[u] + 1, xhi[u], vote >> 4);
                } else {
                    nlo = update_rn4(xlo[u], vote & 0xFu, a.lr, a.wd, has_wd);
                    nhi = update_rn4(xhi[u], vote >> 4, a.lr, a.wd, has_wd);
                }
                __stcs(reinterpret_cast<float4*>(a.x) + 2 * o[u], nlo);
                __stcs(reinterpret_cast<float4*>(a.x) + 2 * o[u] + 1, nhi);
            }
            if (a.words != nullptr) {  // every lane of the warp takes part in the shuffles
                uint32_t w = vote << (8 * k4);
                w |= __shfl_xor_sync(0xFFFFFFFFu, w, 1);
                w |= __shfl_xor_sync(0xFFFFFFFFu, w, 2);
                if (k4 == 0 && ok[u]) a.words[o[u] >> 2] = w;
            }
        }
    }

    // the ragged last word (d not a multiple of 32): one warp, ballot form, run-time worker loop
    if ((a.d & 31) != 0 && blockIdx.x == 0 && threadIdx.x < 32)
        step_word_ballot<(M_CT == 1 ? 1 : 0), S::NP, BF16, MOM, APPLY, SEG>(a, a.d >> 5, lane);
}

template <int M_CT, bool MOM, bool APPLY, bool SEG>
cudaError_t launch_step_oct_inst(const StepDesc& s, cudaStream_t st) {
    using S = OctShape<M_CT, MOM>;
    StepArgs<S::NP> a;
    fill_step_args(a, s, MOM);
    const int threads = launch_threads();
    int grid = 1;
    auto kernel = step_oct_bf16_kernel<M_CT, MOM, APPLY, SEG>;
    const int64_t octets = (s.d >> 5) << 2;
    const int64_t tile = static_cast<int64_t>(threads) * S::U;
    cudaError_t err = pick_grid(kernel, threads, (octets + tile - 1) / tile, &grid);
    if (err != cudaSuccess) return err;
    kernel<<<grid, threads, 0, st>>>(a);
    return cudaGetLastError();
}

// the octet kernels serve every call whose gradient, momentum and parameter pointers are all
// 16-byte aligned; same specialisations of the worker count as the quad form
template <bool SEG>
cudaError_t launch_step_oct(const StepDesc& s, cudaStream_t st) {
    const bool mom = s.v != nullptr;
    if (s.x == nullptr) return launch_step_oct_inst<1, true, false, false>(s, st);  // ss_signum_update
#define SS_OCT_PICK(MV) \
    (mom ? launch_step_oct_inst<MV, true, true, SEG>(s, st) : launch_step_oct_inst<MV, false, true, SEG>(s, st))
    switch (s.M) {
        case 1: return SS_OCT_PICK(1);
        case 3: return SS_OCT_PICK(3);
        case 7: return SS_OCT_PICK(7);
        case 15: return SS_OCT_PICK(15);
        case 16: return SS_OCT_PICK(16);
        case 31: return SS_OCT_PICK(31);
        case 63: return SS_OCT_PICK(63);
        default: return SS_OCT_PICK(0);
    }
#undef SS_OCT_PICK
}

}  // namespace ss
