// Flag-ordered exchange for one worker of Algorithm 1 per GPU: after a worker has stored its
// packed signs into every worker's receive buffer ("push sign(v_m)", done by the kernel that
// produces them), it raises its flag in every worker's flag array; before a worker votes, it waits
// until all M flags in its own array have reached the step's epoch. No collective library call is
// on this path. Stores to a peer are plain stores; nothing is read from a peer; the wait polls the
// worker's own memory only, for a bounded time, and reports who was missing instead of hanging.
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "exchange.cuh"

namespace ss {

int cuda_status_public(cudaError_t e);  // abi.cu

namespace {

struct FlagDests {
    uint32_t* p[SS_MAX_WORKERS];
    int n;
};

// One thread per destination. The kernel runs after the work enqueued before it on the stream has
// completed (all of the push kernel's stores have been performed); the fence orders this thread's
// flag store behind them at system scope for the peer that will read it.
__global__ void flags_signal_kernel(const __grid_constant__ FlagDests dst, int index, uint32_t epoch) {
    const int p = threadIdx.x;
    if (p < dst.n) {
        __threadfence_system();
        *reinterpret_cast<volatile uint32_t*>(dst.p[p] + index) = epoch;
    }
}

// epochs wrap around: a >= b in the sense of serial numbers
__device__ __forceinline__ bool reached(uint32_t a, uint32_t b) { return static_cast<int32_t>(a - b) >= 0; }

// One block. Thread m polls flag m of this GPU's own array until it has reached the epoch, the
// time limit has passed, or the iteration limit has been hit (each round sleeps about a
// microsecond, so the second limit is a multiple of the first and only a backstop). The block
// then writes 0 (every flag arrived) or 1 + the lowest missing worker to *status and returns.
template <bool SIGNAL>
__global__ void flags_wait_kernel(const __grid_constant__ FlagDests dst, int index, const uint32_t* flags,
                                  int M, uint32_t epoch, uint64_t timeout_ns, uint64_t max_rounds,
                                  uint32_t* status) {
    __shared__ int missing;  // lowest worker whose flag never arrived, or INT_MAX
    const int m = threadIdx.x;
    if (m == 0) missing = 0x7FFFFFFF;
    if (SIGNAL && m < dst.n) {  // raise this worker's flag everywhere first (as flags_signal_kernel)
        __threadfence_system();
        *reinterpret_cast<volatile uint32_t*>(dst.p[m] + index) = epoch;
    }
    __syncthreads();
    if (m < M) {
        const volatile uint32_t* f = flags + m;
        uint64_t t0;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
        bool ok = reached(*f, epoch);
        for (uint64_t round = 0; !ok && round < max_rounds; ++round) {
            __nanosleep(1000);
            ok = reached(*f, epoch);
            uint64_t t1;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
            if (t1 - t0 > timeout_ns) {
                ok = ok || reached(*f, epoch);
                break;
            }
        }
        if (!ok) atomicMin(&missing, m);
    }
    __syncthreads();
    if (m == 0) {
        __threadfence_system();  // what the flags announce is read by the kernels that follow
        *status = missing == 0x7FFFFFFF ? 0u : static_cast<uint32_t>(missing) + 1u;
    }
}

inline bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3) == 0; }

}  // namespace
}  // namespace ss

using namespace ss;

extern "C" {
#pragma GCC visibility push(default)

int ss_flags_signal(uint32_t* const* flags, int n_flags, int index, uint32_t epoch, void* cuda_stream) {
    if (flags == nullptr || n_flags < 1 || n_flags > SS_MAX_WORKERS || index < 0 || index >= SS_MAX_WORKERS)
        return SS_ERR_INVALID_ARG;
    FlagDests dst;
    for (int p = 0; p < SS_MAX_WORKERS; ++p) {
        dst.p[p] = p < n_flags ? flags[p] : nullptr;
        if (p < n_flags && flags[p] == nullptr) return SS_ERR_INVALID_ARG;
        if (p < n_flags && !aligned4(flags[p])) return SS_ERR_MISALIGNED;
    }
    dst.n = n_flags;
    flags_signal_kernel<<<1, SS_MAX_WORKERS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(dst, index, epoch);
    return cuda_status_public(cudaGetLastError());
}

int ss_flags_wait(const uint32_t* flags_local, int M, uint32_t epoch, uint64_t timeout_ns,
                  uint32_t* status_dev, void* cuda_stream) {
    if (flags_local == nullptr || status_dev == nullptr || M < 1 || M > SS_MAX_WORKERS)
        return SS_ERR_INVALID_ARG;
    if (timeout_ns > SS_FLAGS_MAX_TIMEOUT_NS) return SS_ERR_INVALID_ARG;
    if (!aligned4(flags_local) || !aligned4(status_dev)) return SS_ERR_MISALIGNED;
    const uint64_t max_rounds = timeout_ns / 250u + 64u;  // >= 4x the time limit in ~1 us rounds
    FlagDests none;
    for (int p = 0; p < SS_MAX_WORKERS; ++p) none.p[p] = nullptr;
    none.n = 0;
    flags_wait_kernel<false><<<1, SS_MAX_WORKERS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        none, 0, flags_local, M, epoch, timeout_ns, max_rounds, status_dev);
    return cuda_status_public(cudaGetLastError());
}

int ss_flags_signal_wait(uint32_t* const* flags, int n_flags, int index, const uint32_t* flags_local, int M,
                         uint32_t epoch, uint64_t timeout_ns, uint32_t* status_dev, void* cuda_stream) {
    if (flags == nullptr || n_flags < 1 || n_flags > SS_MAX_WORKERS || index < 0 || index >= SS_MAX_WORKERS)
        return SS_ERR_INVALID_ARG;
    if (flags_local == nullptr || status_dev == nullptr || M < 1 || M > SS_MAX_WORKERS)
        return SS_ERR_INVALID_ARG;
    if (timeout_ns > SS_FLAGS_MAX_TIMEOUT_NS) return SS_ERR_INVALID_ARG;
    if (!aligned4(flags_local) || !aligned4(status_dev)) return SS_ERR_MISALIGNED;
    FlagDests dst;
    for (int p = 0; p < SS_MAX_WORKERS; ++p) {
        dst.p[p] = p < n_flags ? flags[p] : nullptr;
        if (p < n_flags && flags[p] == nullptr) return SS_ERR_INVALID_ARG;
        if (p < n_flags && !aligned4(flags[p])) return SS_ERR_MISALIGNED;
    }
    dst.n = n_flags;
    const uint64_t max_rounds = timeout_ns / 250u + 64u;
    flags_wait_kernel<true><<<1, SS_MAX_WORKERS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        dst, index, flags_local, M, epoch, timeout_ns, max_rounds, status_dev);
    return cuda_status_public(cudaGetLastError());
}

#pragma GCC visibility pop
}  // extern "C"
