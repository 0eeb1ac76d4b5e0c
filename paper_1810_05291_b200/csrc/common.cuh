// Shared device helpers: streaming loads/stores, the 1-bit sign, and the fp32 arithmetic of
// Algorithm 1 written with explicitly rounded intrinsics so that no multiply-add is fused.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/signsgd.h"

namespace ss {

// Load policies of the streaming kernels. Every byte is touched once, so the natural form is the
// evict-first load (ld.global.cs), and it is the better one for pure read streams (sign packing,
// packed words). In the step kernels, which also write, plain loads (cached at all levels) measure
// faster: same box, same run, fused step, ms per launch, evict-first everywhere / plain for the
// read-modify-write streams only (momenta, parameters) / plain everywhere:
//   M = 15 fp32 Signum (ResNet-50 size)   0.7108 / 0.7034 / 0.6949
//   M = 7 fp32 signSGD (AlexNet size)     0.3179 / 0.3175 / 0.3074
//   M = 15 bf16 Signum, octet kernel      0.6063 / 0.5989 / 0.5940
//   M = 15 fp32 signSGD, d = 2^28         2.6510 / 2.6504 / 2.5375
// with exceptions that keep evict-first gradient loads: the run-time-M kernel without momentum
// (M = 63, d = 2^28: 10.1 ms either way, 18.2 ms with plain gradient loads), calls without
// momentum that read less than 1.5 GiB of gradients (the launcher decides, step_kernel.cuh), and
// the one-worker bf16 momentum update, which keeps evict-first loads throughout (0.0389 against
// 0.0410 ms). The kernels therefore take the policy of their gradient loads as a compile-time
// flag; momenta and parameters are loaded plain (ld_rmw) everywhere else.
template <typename T>
__device__ __forceinline__ T ld_stream(const T* p) {
    return __ldcs(p);
}
template <bool PLAIN, typename T>
__device__ __forceinline__ T ld_grad(const T* p) {
    if constexpr (PLAIN) return *p;
    else return __ldcs(p);
}
template <typename T>
__device__ __forceinline__ T ld_rmw(const T* p) {
    return *p;
}
template <bool PLAIN, typename T>
__device__ __forceinline__ T ld_rmw_as(const T* p) {  // for the one kernel that keeps evict-first throughout
    if constexpr (PLAIN) return *p;
    else return __ldcs(p);
}

struct F32 {
    static constexpr int kBytes = 4;
    // four consecutive coordinates starting at coordinate 4 q
    template <bool PLAIN = false>
    static __device__ __forceinline__ float4 load4(const void* base, int64_t q) {
        return ld_grad<PLAIN>(reinterpret_cast<const float4*>(base) + q);
    }
    static __device__ __forceinline__ float load1(const void* base, int64_t c) {
        return ld_stream(reinterpret_cast<const float*>(base) + c);
    }
};

struct BF16 {
    static constexpr int kBytes = 2;
    template <bool PLAIN = false>
    static __device__ __forceinline__ float4 load4(const void* base, int64_t q) {
        const uint2 r = ld_grad<PLAIN>(reinterpret_cast<const uint2*>(base) + q);
        float4 f;
        f.x = __uint_as_float(r.x << 16);
        f.y = __uint_as_float(r.x & 0xFFFF0000u);
        f.z = __uint_as_float(r.y << 16);
        f.w = __uint_as_float(r.y & 0xFFFF0000u);
        return f;
    }
    static __device__ __forceinline__ float load1(const void* base, int64_t c) {
        const unsigned short h = ld_stream(reinterpret_cast<const unsigned short*>(base) + c);
        return __uint_as_float(static_cast<uint32_t>(h) << 16);
    }
};

// sign(z) as one bit: 1 iff z >= 0 by value (so +-0 -> 1, NaN -> 0).
__device__ __forceinline__ uint32_t sign_bit(float z) { return z >= 0.0f ? 1u : 0u; }

__device__ __forceinline__ uint32_t sign_nibble(const float4& s) {
    return sign_bit(s.x) | (sign_bit(s.y) << 1) | (sign_bit(s.z) << 2) | (sign_bit(s.w) << 3);
}

// v <- (1 - beta) g + beta v: two rounded multiplies, one rounded add (Algorithm 1, momentum).
__device__ __forceinline__ float momentum_rn(float omb, float g, float beta, float v) {
    return __fadd_rn(__fmul_rn(omb, g), __fmul_rn(beta, v));
}

__device__ __forceinline__ float4 momentum_rn4(float omb, const float4& g, float beta,
                                               const float4& v) {
    float4 r;
    r.x = momentum_rn(omb, g.x, beta, v.x);
    r.y = momentum_rn(omb, g.y, beta, v.y);
    r.z = momentum_rn(omb, g.z, beta, v.z);
    r.w = momentum_rn(omb, g.w, beta, v.w);
    return r;
}

// x <- x - lr (s + wd x), s = +1 if plus else -1 (Algorithm 1, parameter update).
__device__ __forceinline__ float update_rn(float x, uint32_t plus, float lr, float wd,
                                           bool has_wd) {
    if (!has_wd) return __fsub_rn(x, plus ? lr : -lr);
    const float s = plus ? 1.0f : -1.0f;
    return __fsub_rn(x, __fmul_rn(lr, __fadd_rn(s, __fmul_rn(wd, x))));
}

__device__ __forceinline__ float4 update_rn4(const float4& x, uint32_t nib, float lr, float wd,
                                             bool has_wd) {
    float4 r;
    r.x = update_rn(x.x, nib & 1u, lr, wd, has_wd);
    r.y = update_rn(x.y, nib & 2u, lr, wd, has_wd);
    r.z = update_rn(x.z, nib & 4u, lr, wd, has_wd);
    r.w = update_rn(x.w, nib & 8u, lr, wd, has_wd);
    return r;
}

// ---- per-tensor hyper-parameters of a fused flat vector (Section 4: small tensors are merged
// into one buffer before compression). The table is sorted by first coordinate; entry k covers
// [begin_k, begin_{k+1}) and the last entry runs to d. -------------------------------------------

// index of the last entry whose begin is <= c (entry 0 begins at coordinate 0)
__device__ __forceinline__ int segment_of(const ss_segment* seg, int n, int64_t c) {
    int lo = 0, hi = n;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(&seg[mid].begin) <= c) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ float update_seg1(const ss_segment* seg, int n, int64_t c, float x,
                                             uint32_t plus) {
    const int k = segment_of(seg, n, c);
    const float lr = __ldg(&seg[k].lr), wd = __ldg(&seg[k].weight_decay);
    return update_rn(x, plus, lr, wd, wd != 0.0f);
}

// the quad of coordinates 4 q .. 4 q + 3: one lookup when the quad lies inside one tensor
__device__ __forceinline__ float4 update_seg4(const ss_segment* seg, int n, int64_t q,
                                              const float4& x, uint32_t nib) {
    const int64_t c0 = q << 2;
    const int k = segment_of(seg, n, c0);
    const bool whole = (k + 1 >= n) || (__ldg(&seg[k + 1].begin) > c0 + 3);
    if (whole) {
        const float lr = __ldg(&seg[k].lr), wd = __ldg(&seg[k].weight_decay);
        return update_rn4(x, nib, lr, wd, wd != 0.0f);
    }
    float4 r;
    r.x = update_seg1(seg, n, c0, x.x, nib & 1u);
    r.y = update_seg1(seg, n, c0 + 1, x.y, nib & 2u);
    r.z = update_seg1(seg, n, c0 + 2, x.z, nib & 4u);
    r.w = update_seg1(seg, n, c0 + 3, x.w, nib & 8u);
    return r;
}

// ---- host side --------------------------------------------------------------------------

// Launch-shape overrides (ss_set_launch_option): process-wide, read atomically at every launch.
constexpr int kMaxBlockThreads = 256;  // every kernel is compiled with __launch_bounds__(256)
int launch_threads();        // block size to use: the "threads" option, or 256 when it is 0
int launch_blocks_per_sm();  // 0: one block per tile; > 0: persistent grid of this many blocks per SM
int64_t launch_plain_loads_from_bytes();  // gradient bytes per call from which the unrolled kernels
                                          // without momentum load the gradients plain (see ld_grad)
int device_sm_count(cudaError_t* err);

// Grid size for a grid-stride kernel. Default: one block per tile. On B200 the hardware block
// scheduler feeding short-lived blocks sustains a higher HBM rate than a persistent grid whose
// blocks stride in lock step (fused Signum step, M = 15: 6.8 TB/s against 6.2 TB/s), so the
// persistent form (blocks_per_sm blocks per SM) is kept only as a launch option.
template <typename Kernel>
inline cudaError_t pick_grid(Kernel kernel, int threads, int64_t blocks_needed, int* grid_out) {
    (void)kernel;
    int64_t grid = blocks_needed;
    const int per_sm = launch_blocks_per_sm();
    if (per_sm > 0) {
        cudaError_t err = cudaSuccess;
        const int sms = device_sm_count(&err);
        if (err != cudaSuccess) return err;
        const int64_t persistent = static_cast<int64_t>(sms) * per_sm;
        if (grid > persistent) grid = persistent;
    }
    if (grid > 0x7FFFFFFFll) grid = 0x7FFFFFFFll;
    if (grid < 1) grid = 1;
    *grid_out = static_cast<int>(grid);
    return cudaSuccess;
}

// ---- launch descriptors (filled by the C ABI after validation) ------------------------------

struct StepDesc {
    const void* const* g;   // M device pointers (host array)
    float* const* v;        // M device pointers (host array) or null
    int M;
    int64_t d;
    float beta, omb, lr, wd;
    uint64_t flip;
    float* x;               // null: no parameter update (pack only)
    uint32_t* words;        // may be null when x != null
    bool vec;               // all pointers sufficiently aligned for 128-bit access
    const ss_segment* seg = nullptr;  // device table of per-tensor lr / weight decay, or null
    int n_seg = 0;
};

// abi.cu: every argument check of a step, with no CUDA call (on SS_OK *out describes the launch;
// out->d == 0 means nothing to do), and the launch of a checked step
int validate_step(const void* const* grads, ss_dtype dt, float* const* momenta, int M, int64_t d,
                  float beta, uint64_t flip_mask, float* param, float lr, float weight_decay,
                  uint32_t* words, const ss_segment* seg, int n_seg, StepDesc* out);
int launch_step(const StepDesc& s, ss_dtype dt, void* cuda_stream);

cudaError_t launch_step_f32(const StepDesc& s, cudaStream_t st);
cudaError_t launch_step_bf16(const StepDesc& s, cudaStream_t st);
cudaError_t launch_signum_push_f32(const void* g, float* v, float beta, float omb, int64_t d,
                                   uint32_t* const* dests, int n, bool vec, cudaStream_t st);
cudaError_t launch_signum_push_bf16(const void* g, float* v, float beta, float omb, int64_t d,
                                    uint32_t* const* dests, int n, bool vec, cudaStream_t st);
cudaError_t launch_vote(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                        uint32_t* vote, bool vec, cudaStream_t st);
cudaError_t launch_vote_apply(const uint32_t* const* packed, int M, int64_t d, uint64_t flip,
                              float* x, float lr, float wd, bool vec, const ss_segment* seg,
                              int n_seg, uint32_t* vote, cudaStream_t st);
cudaError_t launch_tally(const uint32_t* const* packed, int M, int64_t d, uint64_t flip, int8_t* out,
                         cudaStream_t st);
cudaError_t launch_apply(float* x, const uint32_t* vote, int64_t d, float lr, float wd, bool vec,
                         const ss_segment* seg, int n_seg, cudaStream_t st);

}  // namespace ss
