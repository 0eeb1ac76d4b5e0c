// ss_fused_step_host_static: the host-gradient step for callers that cannot allocate device
// memory. Its staging area is a fixed array that is part of this library's device image.
#include <cuda_runtime.h>

#include <mutex>

#include "common.cuh"

namespace ss {
int cuda_status_public(cudaError_t e);  // abi.cu: records the error for ss_last_cuda_error()
}

// The staging area. It exists once per GPU that loads this library, from the moment the CUDA
// module is loaded until the process exits, whether or not the entry point is ever called.
static __device__ __align__(256) unsigned char g_static_staging[SS_STATIC_STAGING_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
unsigned char* g_staging_addr[kMaxDevices] = {nullptr};

// In host code `g_static_staging` is only a handle for the runtime, not an address a kernel or
// a copy may use. The device address has to be asked for, once per device, with that device
// current; it is then kept for the life of the process.
cudaError_t staging_for_current_device(unsigned char** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_staging_addr[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_staging);
        if (e != cudaSuccess) return e;
        if (p == nullptr) return cudaErrorInvalidSymbol;
        g_staging_addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_staging_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

int ss_fused_step_host_static(const void* const* host_grads, ss_dtype dt, float* const* momenta,
                              int M, int64_t d, float beta, uint64_t flip_mask, float* param,
                              float lr, float weight_decay, uint32_t* vote_words_dev,
                              uint32_t* host_vote_out, void* cuda_stream) {
    if ((dt != SS_F32 && dt != SS_BF16) || M < 1 || M > SS_MAX_WORKERS || d < 0 || d > SS_MAX_COORDS)
        return SS_ERR_INVALID_ARG;
    if (M < 64 && (flip_mask >> M) != 0) return SS_ERR_INVALID_ARG;
    if (d == 0) return SS_OK;
    if (host_grads == nullptr || param == nullptr || vote_words_dev == nullptr) return SS_ERR_INVALID_ARG;
    for (int m = 0; m < M; ++m)
        if (host_grads[m] == nullptr) return SS_ERR_INVALID_ARG;

    // worker m's gradients are staged at m * slot, slots rounded up to 256 bytes. The limit is
    // tested by division, before any product is formed, so that no d can wrap the byte counts.
    const uint64_t es = dt == SS_F32 ? 4u : 2u;
    const uint64_t cap = SS_STATIC_STAGING_BYTES;
    if (static_cast<uint64_t>(d) > cap / es) return SS_ERR_UNSUPPORTED;
    const uint64_t gbytes = static_cast<uint64_t>(d) * es;
    const uint64_t slot = (gbytes + 255u) & ~static_cast<uint64_t>(255u);
    if (slot > cap / static_cast<uint64_t>(M)) return SS_ERR_UNSUPPORTED;  // M * slot > the fixed area

    // First pass over the caller's own pointers (alignment, NULL entries, overlaps among momenta,
    // param and the vote buffer), with the host gradients standing in for the staged ones: argument
    // errors are reported before any CUDA call.
    ss::StepDesc step;
    int rc = ss::validate_step(host_grads, dt, momenta, M, d, beta, flip_mask, param, lr, weight_decay,
                               vote_words_dev, nullptr, 0, &step);
    if (rc != SS_OK) return rc;

    unsigned char* base = nullptr;
    cudaError_t e = staging_for_current_device(&base);
    if (e != cudaSuccess) return ss::cuda_status_public(e);

    // the whole step is checked against the staged addresses before the first copy is enqueued
    const void* staged[SS_MAX_WORKERS];
    for (int m = 0; m < M; ++m) staged[m] = base + slot * static_cast<uint64_t>(m);
    rc = ss::validate_step(staged, dt, momenta, M, d, beta, flip_mask, param, lr, weight_decay,
                           vote_words_dev, nullptr, 0, &step);
    if (rc != SS_OK) return rc;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    for (int m = 0; m < M; ++m) {
        e = cudaMemcpyAsync(const_cast<void*>(staged[m]), host_grads[m], gbytes, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return ss::cuda_status_public(e);
    }
    const int lrc = ss::launch_step(step, dt, cuda_stream);
    if (lrc != SS_OK) return lrc;
    if (host_vote_out != nullptr) {
        e = cudaMemcpyAsync(host_vote_out, vote_words_dev, static_cast<size_t>((d + 31) / 32) * 4,
                            cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return ss::cuda_status_public(e);
    }
    return SS_OK;
}

#pragma GCC visibility pop
}  // extern "C"
