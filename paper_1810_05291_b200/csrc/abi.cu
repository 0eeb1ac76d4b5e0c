// The C ABI: argument validation, alignment classification and kernel dispatch. Every step of
// the path runs in the kernels; nothing here touches the data.
#include <atomic>
#include <cstring>

#include "common.cuh"
#include "exchange.cuh"

namespace ss {

namespace {
std::atomic<int> g_opt_threads{0};
std::atomic<int> g_opt_blocks_per_sm{0};
std::atomic<int> g_opt_plain_from_mib{0};
constexpr int kDefaultPlainFromMib = 1536;
}  // namespace

int launch_threads() {
    const int t = g_opt_threads.load(std::memory_order_relaxed);
    return t > 0 ? t : kMaxBlockThreads;
}

int launch_blocks_per_sm() { return g_opt_blocks_per_sm.load(std::memory_order_relaxed); }

int64_t launch_plain_loads_from_bytes() {
    const int mib = g_opt_plain_from_mib.load(std::memory_order_relaxed);
    return static_cast<int64_t>(mib > 0 ? mib : kDefaultPlainFromMib) << 20;
}

int device_sm_count(cudaError_t* err) {
    static int cached[64] = {0};
    int dev = 0;
    *err = cudaGetDevice(&dev);
    if (*err != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64 && cached[dev] > 0) return cached[dev];
    int sms = 0;
    *err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (*err != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64) cached[dev] = sms;
    return sms;
}

namespace {

thread_local int t_last_cuda_error = 0;

int cuda_status(cudaError_t e) {
    if (e == cudaSuccess) return SS_OK;
    t_last_cuda_error = static_cast<int>(e);
    return SS_ERR_CUDA;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

inline int elem_bytes(ss_dtype dt) { return dt == SS_F32 ? 4 : 2; }

inline bool dtype_ok(ss_dtype dt) { return dt == SS_F32 || dt == SS_BF16; }

inline bool flip_ok(uint64_t flip, int M) { return M >= 64 || (flip >> M) == 0; }

// 0 <= d <= SS_MAX_COORDS: keeps every byte count formed from d far inside 64 bits
inline bool d_ok(int64_t d) { return d >= 0 && d <= SS_MAX_COORDS; }

// half-open byte ranges [p, p + n)
inline bool overlap(const void* p, size_t n, const void* q, size_t m) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(p), b = reinterpret_cast<uintptr_t>(q);
    return n != 0 && m != 0 && a < b + m && b < a + n;
}

}  // namespace

// for the other translation units of the library
int cuda_status_public(cudaError_t e) { return cuda_status(e); }

}  // namespace ss

namespace ss {

// Every check of a step's arguments, with no CUDA call and nothing enqueued. On SS_OK *out
// describes the launch (out->d == 0: nothing to do).
int validate_step(const void* const* grads, ss_dtype dt, float* const* momenta, int M, int64_t d,
                  float beta, uint64_t flip_mask, float* param, float lr, float weight_decay,
                  uint32_t* words, const ss_segment* seg, int n_seg, StepDesc* out) {
    if (!dtype_ok(dt) || M < 1 || M > SS_MAX_WORKERS || !d_ok(d)) return SS_ERR_INVALID_ARG;
    if (!flip_ok(flip_mask, M)) return SS_ERR_INVALID_ARG;
    out->d = 0;
    if (d == 0) return SS_OK;
    if (grads == nullptr || (param == nullptr && words == nullptr)) return SS_ERR_INVALID_ARG;
    const size_t eb = static_cast<size_t>(elem_bytes(dt));
    const size_t gbytes = static_cast<size_t>(d) * eb, fbytes = static_cast<size_t>(d) * 4;
    const size_t wbytes = static_cast<size_t>((d + 31) / 32) * 4;
    bool vec = true;
    for (int m = 0; m < M; ++m) {
        if (grads[m] == nullptr) return SS_ERR_INVALID_ARG;
        if (!aligned(grads[m], eb)) return SS_ERR_MISALIGNED;
        vec = vec && aligned(grads[m], eb * 4);
        if (param != nullptr && overlap(grads[m], gbytes, param, fbytes)) return SS_ERR_INVALID_ARG;
        if (words != nullptr && overlap(grads[m], gbytes, words, wbytes)) return SS_ERR_INVALID_ARG;
    }
    if (momenta != nullptr) {
        for (int m = 0; m < M; ++m) {
            if (momenta[m] == nullptr) return SS_ERR_INVALID_ARG;
            if (!aligned(momenta[m], 4)) return SS_ERR_MISALIGNED;
            vec = vec && aligned(momenta[m], 16);
            if (param != nullptr && overlap(momenta[m], fbytes, param, fbytes)) return SS_ERR_INVALID_ARG;
            if (words != nullptr && overlap(momenta[m], fbytes, words, wbytes)) return SS_ERR_INVALID_ARG;
            for (int k = 0; k < M; ++k)  // a momentum buffer is written: it may alias no gradient
                if (overlap(momenta[m], fbytes, grads[k], gbytes)) return SS_ERR_INVALID_ARG;
            for (int k = 0; k < m; ++k)
                if (overlap(momenta[m], fbytes, momenta[k], fbytes)) return SS_ERR_INVALID_ARG;
        }
    }
    if (param != nullptr) {
        if (!aligned(param, 4)) return SS_ERR_MISALIGNED;
        vec = vec && aligned(param, 16);
        if (words != nullptr && overlap(param, fbytes, words, wbytes)) return SS_ERR_INVALID_ARG;
    }
    if (words != nullptr && !aligned(words, 4)) return SS_ERR_MISALIGNED;

    StepDesc& s = *out;
    s.g = grads;
    s.v = momenta;
    s.M = M;
    s.d = d;
    s.beta = momenta != nullptr ? beta : 0.0f;
    s.omb = 1.0f - s.beta;
    s.lr = lr;
    s.wd = weight_decay;
    s.flip = flip_mask;
    s.x = param;
    s.words = words;
    s.vec = vec;
    s.seg = seg;
    s.n_seg = n_seg;
    return SS_OK;
}

int launch_step(const StepDesc& s, ss_dtype dt, void* cuda_stream) {
    if (s.d == 0) return SS_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    return cuda_status(dt == SS_F32 ? launch_step_f32(s, st) : launch_step_bf16(s, st));
}

}  // namespace ss


using namespace ss;

extern "C" {
#pragma GCC visibility push(default)

int64_t ss_packed_words(int64_t d) { return d < 0 ? -1 : (d + 31) / 32; }

const char* ss_status_string(int status) {
    switch (status) {
        case SS_OK: return "SS_OK";
        case SS_ERR_INVALID_ARG: return "SS_ERR_INVALID_ARG: null pointer, size or worker count out of range, or flip_mask bit >= M";
        case SS_ERR_MISALIGNED: return "SS_ERR_MISALIGNED: pointer not aligned to its element size";
        case SS_ERR_UNSUPPORTED: return "SS_ERR_UNSUPPORTED: request not served by this build";
        case SS_ERR_CUDA: return "SS_ERR_CUDA: CUDA runtime or launch failure (see ss_last_cuda_error)";
        default: return "unknown status";
    }
}

int ss_last_cuda_error(void) { return t_last_cuda_error; }

int ss_set_launch_option(const char* key, int value) {
    if (key == nullptr) return SS_ERR_INVALID_ARG;
    if (std::strcmp(key, "threads") == 0) {
        if (value != 0 && (value < 64 || value > kMaxBlockThreads || (value & 31) != 0))
            return SS_ERR_INVALID_ARG;
        g_opt_threads.store(value, std::memory_order_relaxed);
        return SS_OK;
    }
    if (std::strcmp(key, "plain_loads_from_mib") == 0) {
        if (value < 0 || value > (1 << 20)) return SS_ERR_INVALID_ARG;
        g_opt_plain_from_mib.store(value, std::memory_order_relaxed);
        return SS_OK;
    }
    if (std::strcmp(key, "blocks_per_sm") == 0) {
        if (value < 0 || value > 4096) return SS_ERR_INVALID_ARG;
        g_opt_blocks_per_sm.store(value, std::memory_order_relaxed);
        return SS_OK;
    }
    return SS_ERR_INVALID_ARG;
}

static int step_common(const void* const* grads, ss_dtype dt, float* const* momenta, int M,
                       int64_t d, float beta, uint64_t flip_mask, float* param, float lr,
                       float weight_decay, uint32_t* words, void* cuda_stream,
                       const ss_segment* seg = nullptr, int n_seg = 0) {
    StepDesc s;
    const int rc = validate_step(grads, dt, momenta, M, d, beta, flip_mask, param, lr, weight_decay,
                                 words, seg, n_seg, &s);
    return rc != SS_OK ? rc : launch_step(s, dt, cuda_stream);
}

int ss_sign_pack(const void* grad, ss_dtype dt, int64_t d, uint32_t* out_words, void* cuda_stream) {
    if (d > 0 && (grad == nullptr || out_words == nullptr)) return SS_ERR_INVALID_ARG;
    const void* g[1] = {grad};
    return step_common(g, dt, nullptr, 1, d, 0.0f, 0, nullptr, 0.0f, 0.0f, out_words, cuda_stream);
}

int ss_signum_update(const void* grad, ss_dtype dt, float* momentum, float beta, int64_t d,
                     uint32_t* out_words, void* cuda_stream) {
    if (d > 0 && (grad == nullptr || momentum == nullptr || out_words == nullptr)) return SS_ERR_INVALID_ARG;
    const void* g[1] = {grad};
    float* v[1] = {momentum};
    return step_common(g, dt, v, 1, d, beta, 0, nullptr, 0.0f, 0.0f, out_words, cuda_stream);
}

int ss_signum_update_push(const void* grad, ss_dtype dt, float* momentum, float beta, int64_t d,
                          uint32_t* const* dests, int n_dests, void* cuda_stream) {
    if (!dtype_ok(dt) || !d_ok(d) || n_dests < 1 || n_dests > SS_MAX_WORKERS) return SS_ERR_INVALID_ARG;
    if (d == 0) return SS_OK;
    if (grad == nullptr || momentum == nullptr || dests == nullptr) return SS_ERR_INVALID_ARG;
    const size_t eb = static_cast<size_t>(elem_bytes(dt));
    const size_t gbytes = static_cast<size_t>(d) * eb, fbytes = static_cast<size_t>(d) * 4;
    const size_t wbytes = static_cast<size_t>((d + 31) / 32) * 4;
    if (!aligned(grad, eb) || !aligned(momentum, 4)) return SS_ERR_MISALIGNED;
    if (overlap(grad, gbytes, momentum, fbytes)) return SS_ERR_INVALID_ARG;
    for (int p = 0; p < n_dests; ++p) {
        if (dests[p] == nullptr) return SS_ERR_INVALID_ARG;
        if (!aligned(dests[p], 4)) return SS_ERR_MISALIGNED;
        if (overlap(dests[p], wbytes, momentum, fbytes) || overlap(dests[p], wbytes, grad, gbytes))
            return SS_ERR_INVALID_ARG;
        for (int q = 0; q < p; ++q)
            if (overlap(dests[p], wbytes, dests[q], wbytes)) return SS_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // off the 16-byte grid the ballot-form kernel runs; it stores to every destination as well
    const bool vec = aligned(grad, eb * 4) && aligned(momentum, 16);
    const float omb = 1.0f - beta;
    return cuda_status(dt == SS_F32
                           ? launch_signum_push_f32(grad, momentum, beta, omb, d, dests, n_dests, vec, st)
                           : launch_signum_push_bf16(grad, momentum, beta, omb, d, dests, n_dests, vec, st));
}

int ss_fused_step(const void* const* grads, ss_dtype dt, float* const* momenta, int M, int64_t d,
                  float beta, uint64_t flip_mask, float* param, float lr, float weight_decay,
                  uint32_t* vote_words_out, void* cuda_stream) {
    if (d > 0 && param == nullptr) return SS_ERR_INVALID_ARG;
    return step_common(grads, dt, momenta, M, d, beta, flip_mask, param, lr, weight_decay,
                       vote_words_out, cuda_stream);
}

int ss_majority_vote(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                     uint32_t* vote_words, void* cuda_stream) {
    if (packed == nullptr || M < 1 || M > SS_MAX_WORKERS || !d_ok(d)) return SS_ERR_INVALID_ARG;
    if (!flip_ok(flip_mask, M)) return SS_ERR_INVALID_ARG;
    if (d == 0) return SS_OK;
    if (vote_words == nullptr) return SS_ERR_INVALID_ARG;
    if (!aligned(vote_words, 4)) return SS_ERR_MISALIGNED;
    const size_t wbytes = static_cast<size_t>((d + 31) / 32) * 4;
    bool vec = aligned(vote_words, 16);
    for (int m = 0; m < M; ++m) {
        if (packed[m] == nullptr) return SS_ERR_INVALID_ARG;
        if (!aligned(packed[m], 4)) return SS_ERR_MISALIGNED;
        if (overlap(packed[m], wbytes, vote_words, wbytes)) return SS_ERR_INVALID_ARG;
        vec = vec && aligned(packed[m], 16);
    }
    return cuda_status(launch_vote(packed, M, d, flip_mask, vote_words, vec,
                                   static_cast<cudaStream_t>(cuda_stream)));
}

int ss_vote_tally(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                  int8_t* tally_out, void* cuda_stream) {
    if (packed == nullptr || M < 1 || M > SS_MAX_WORKERS || !d_ok(d)) return SS_ERR_INVALID_ARG;
    if (!flip_ok(flip_mask, M)) return SS_ERR_INVALID_ARG;
    if (d == 0) return SS_OK;
    if (tally_out == nullptr) return SS_ERR_INVALID_ARG;
    const size_t wbytes = static_cast<size_t>((d + 31) / 32) * 4;
    for (int m = 0; m < M; ++m) {
        if (packed[m] == nullptr) return SS_ERR_INVALID_ARG;
        if (!aligned(packed[m], 4)) return SS_ERR_MISALIGNED;
        if (overlap(packed[m], wbytes, tally_out, static_cast<size_t>(d))) return SS_ERR_INVALID_ARG;
    }
    return cuda_status(launch_tally(packed, M, d, flip_mask, tally_out,
                                    static_cast<cudaStream_t>(cuda_stream)));
}

int ss_apply_vote(float* param, const uint32_t* vote_words, int64_t d, float lr, float weight_decay,
                  void* cuda_stream) {
    if (!d_ok(d)) return SS_ERR_INVALID_ARG;
    if (d == 0) return SS_OK;
    if (param == nullptr || vote_words == nullptr) return SS_ERR_INVALID_ARG;
    if (!aligned(param, 4) || !aligned(vote_words, 4)) return SS_ERR_MISALIGNED;
    if (overlap(param, static_cast<size_t>(d) * 4, vote_words, static_cast<size_t>((d + 31) / 32) * 4))
        return SS_ERR_INVALID_ARG;
    return cuda_status(launch_apply(param, vote_words, d, lr, weight_decay, aligned(param, 16),
                                    nullptr, 0, static_cast<cudaStream_t>(cuda_stream)));
}

static int vote_apply_common(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                             float* param, float lr, float weight_decay, const ss_segment* seg,
                             int n_seg, uint32_t* vote_words_out, void* cuda_stream,
                             const uint32_t* guard = nullptr) {
    if (packed == nullptr || M < 1 || M > SS_MAX_WORKERS || !d_ok(d)) return SS_ERR_INVALID_ARG;
    if (!flip_ok(flip_mask, M)) return SS_ERR_INVALID_ARG;
    if (d == 0) return SS_OK;
    if (param == nullptr) return SS_ERR_INVALID_ARG;
    if (!aligned(param, 4)) return SS_ERR_MISALIGNED;
    const size_t wbytes = static_cast<size_t>((d + 31) / 32) * 4, fbytes = static_cast<size_t>(d) * 4;
    if (vote_words_out != nullptr) {
        if (!aligned(vote_words_out, 4)) return SS_ERR_MISALIGNED;
        if (overlap(vote_words_out, wbytes, param, fbytes)) return SS_ERR_INVALID_ARG;
    }
    for (int m = 0; m < M; ++m) {
        if (packed[m] == nullptr) return SS_ERR_INVALID_ARG;
        if (!aligned(packed[m], 4)) return SS_ERR_MISALIGNED;
        if (overlap(packed[m], wbytes, param, fbytes)) return SS_ERR_INVALID_ARG;
        if (vote_words_out != nullptr && overlap(packed[m], wbytes, vote_words_out, wbytes))
            return SS_ERR_INVALID_ARG;
    }
    return cuda_status(launch_vote_apply_guarded(packed, M, d, flip_mask, param, lr, weight_decay,
                                                 aligned(param, 16), seg, n_seg, vote_words_out, guard,
                                                 static_cast<cudaStream_t>(cuda_stream)));
}

// the guard word is read while the call writes: it may lie in neither output
static int guard_ok(const uint32_t* guard, int64_t d, const float* param, const uint32_t* vote_words_out) {
    if (guard == nullptr) return SS_ERR_INVALID_ARG;
    if (!aligned(guard, 4)) return SS_ERR_MISALIGNED;
    if (d > 0 && d_ok(d)) {
        if (param != nullptr && overlap(guard, 4, param, static_cast<size_t>(d) * 4)) return SS_ERR_INVALID_ARG;
        if (vote_words_out != nullptr && overlap(guard, 4, vote_words_out, static_cast<size_t>((d + 31) / 32) * 4))
            return SS_ERR_INVALID_ARG;
    }
    return SS_OK;
}

int ss_vote_apply_guarded(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                          float* param, float lr, float weight_decay, uint32_t* vote_words_out,
                          const uint32_t* skip_if_nonzero_dev, void* cuda_stream) {
    const int rc = guard_ok(skip_if_nonzero_dev, d, param, vote_words_out);
    if (rc != SS_OK) return rc;
    return vote_apply_common(packed, M, d, flip_mask, param, lr, weight_decay, nullptr, 0,
                             vote_words_out, cuda_stream, skip_if_nonzero_dev);
}

int ss_vote_apply_guarded_segments(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                                   float* param, const ss_segment* segments_dev, int n_segments,
                                   uint32_t* vote_words_out, const uint32_t* skip_if_nonzero_dev,
                                   void* cuda_stream) {
    const int rc = guard_ok(skip_if_nonzero_dev, d, param, vote_words_out);
    if (rc != SS_OK) return rc;
    if (n_segments < 1) return SS_ERR_INVALID_ARG;
    if (d > 0 && segments_dev == nullptr) return SS_ERR_INVALID_ARG;
    if (d > 0 && !aligned(segments_dev, 8)) return SS_ERR_MISALIGNED;
    return vote_apply_common(packed, M, d, flip_mask, param, 0.0f, 0.0f, segments_dev, n_segments,
                             vote_words_out, cuda_stream, skip_if_nonzero_dev);
}

int ss_vote_apply(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask, float* param,
                  float lr, float weight_decay, uint32_t* vote_words_out, void* cuda_stream) {
    return vote_apply_common(packed, M, d, flip_mask, param, lr, weight_decay, nullptr, 0,
                             vote_words_out, cuda_stream);
}

int ss_vote_apply_segments(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                           float* param, const ss_segment* segments_dev, int n_segments,
                           uint32_t* vote_words_out, void* cuda_stream) {
    if (n_segments < 1) return SS_ERR_INVALID_ARG;
    if (d > 0 && segments_dev == nullptr) return SS_ERR_INVALID_ARG;
    if (d > 0 && !aligned(segments_dev, 8)) return SS_ERR_MISALIGNED;
    return vote_apply_common(packed, M, d, flip_mask, param, 0.0f, 0.0f, segments_dev, n_segments,
                             vote_words_out, cuda_stream);
}

int ss_segments_upload(const ss_segment* host_segments, int n_segments, int64_t d,
                       ss_segment* segments_dev, void* cuda_stream) {
    if (host_segments == nullptr || segments_dev == nullptr || n_segments < 1 || !d_ok(d))
        return SS_ERR_INVALID_ARG;
    if (!aligned(segments_dev, 8)) return SS_ERR_MISALIGNED;
    if (host_segments[0].begin != 0) return SS_ERR_INVALID_ARG;
    for (int k = 0; k < n_segments; ++k) {
        if (host_segments[k].begin > d) return SS_ERR_INVALID_ARG;
        if (k > 0 && host_segments[k].begin < host_segments[k - 1].begin) return SS_ERR_INVALID_ARG;
    }
    return cuda_status(cudaMemcpyAsync(segments_dev, host_segments,
                                       static_cast<size_t>(n_segments) * sizeof(ss_segment),
                                       cudaMemcpyHostToDevice, static_cast<cudaStream_t>(cuda_stream)));
}

int ss_fused_step_segments(const void* const* grads, ss_dtype dt, float* const* momenta, int M,
                           int64_t d, float beta, uint64_t flip_mask, float* param,
                           const ss_segment* segments_dev, int n_segments,
                           uint32_t* vote_words_out, void* cuda_stream) {
    if (n_segments < 1) return SS_ERR_INVALID_ARG;
    if (d > 0 && (param == nullptr || segments_dev == nullptr)) return SS_ERR_INVALID_ARG;
    if (d > 0 && !aligned(segments_dev, 8)) return SS_ERR_MISALIGNED;
    return step_common(grads, dt, momenta, M, d, beta, flip_mask, param, 0.0f, 0.0f, vote_words_out,
                       cuda_stream, segments_dev, n_segments);
}

int ss_apply_vote_segments(float* param, const uint32_t* vote_words, int64_t d,
                           const ss_segment* segments_dev, int n_segments, void* cuda_stream) {
    if (!d_ok(d) || n_segments < 1) return SS_ERR_INVALID_ARG;
    if (d == 0) return SS_OK;
    if (param == nullptr || vote_words == nullptr || segments_dev == nullptr) return SS_ERR_INVALID_ARG;
    if (!aligned(param, 4) || !aligned(vote_words, 4) || !aligned(segments_dev, 8)) return SS_ERR_MISALIGNED;
    if (overlap(param, static_cast<size_t>(d) * 4, vote_words, static_cast<size_t>((d + 31) / 32) * 4))
        return SS_ERR_INVALID_ARG;
    return cuda_status(launch_apply(param, vote_words, d, 0.0f, 0.0f, aligned(param, 16), segments_dev,
                                    n_segments, static_cast<cudaStream_t>(cuda_stream)));
}

int ss_fused_step_host(const void* const* host_grads, ss_dtype dt, void* const* staging,
                       float* const* momenta, int M, int64_t d, float beta, uint64_t flip_mask,
                       float* param, float lr, float weight_decay, uint32_t* vote_words_dev,
                       uint32_t* host_vote_out, void* cuda_stream) {
    if (!dtype_ok(dt) || M < 1 || M > SS_MAX_WORKERS || !d_ok(d) || !flip_ok(flip_mask, M))
        return SS_ERR_INVALID_ARG;
    if (d == 0) return SS_OK;
    if (host_grads == nullptr || staging == nullptr || vote_words_dev == nullptr || param == nullptr)
        return SS_ERR_INVALID_ARG;
    for (int m = 0; m < M; ++m)
        if (host_grads[m] == nullptr) return SS_ERR_INVALID_ARG;
    // the whole step is checked, with the staging buffers in the gradients' place, before the
    // first copy is enqueued
    StepDesc s;
    const int rc = validate_step(reinterpret_cast<const void* const*>(staging), dt, momenta, M, d, beta,
                                 flip_mask, param, lr, weight_decay, vote_words_dev, nullptr, 0, &s);
    if (rc != SS_OK) return rc;
    const size_t gbytes = static_cast<size_t>(d) * static_cast<size_t>(elem_bytes(dt));
    for (int m = 0; m < M; ++m)  // staging buffers are written: no two may overlap
        for (int k = 0; k < m; ++k)
            if (overlap(staging[m], gbytes, staging[k], gbytes)) return SS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    for (int m = 0; m < M; ++m) {
        cudaError_t e = cudaMemcpyAsync(staging[m], host_grads[m], gbytes, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return cuda_status(e);
    }
    const int lrc = launch_step(s, dt, cuda_stream);
    if (lrc != SS_OK) return lrc;
    if (host_vote_out != nullptr) {
        cudaError_t e = cudaMemcpyAsync(host_vote_out, vote_words_dev,
                                        static_cast<size_t>((d + 31) / 32) * 4, cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return cuda_status(e);
    }
    return SS_OK;
}

#pragma GCC visibility pop
}  // extern "C"
