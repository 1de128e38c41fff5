// C ABI of the library: argument validation on the host, dispatch to the kernels.
#include "../../include/sfda.h"

#include <mutex>

#include "sfda_internal.h"

namespace {

thread_local int g_last_launches = 0;

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_dims(int d_k, int d_v, int chunk, int dtype)
{
    if (d_k < 2 || (d_k & 1) || d_v < 1 || chunk < 1) return SFDA_ERR_SHAPE;
    if (d_k != 64 && d_k != 128) return SFDA_ERR_UNSUPPORTED;
    if (d_v != 64 && d_v != 128) return SFDA_ERR_UNSUPPORTED;
    if (chunk != 16 && chunk != 32 && chunk != 64 && chunk != 128 && chunk != 256) return SFDA_ERR_UNSUPPORTED;
    if (dtype != SFDA_F32 && dtype != SFDA_BF16) return SFDA_ERR_UNSUPPORTED;
    return SFDA_OK;
}

size_t elem_bytes(int dtype) { return dtype == SFDA_BF16 ? 2 : 4; }

// The kernels' tile is at most 64 tokens (tensor memory and shared memory are full at 64).  A chunk of 128 or 256
// tokens is run as an exact superchunk of two or four tiles (Section 6, "superchunks": chunk transfers compose
// exactly): the state is carried on chip from tile to tile, and since the recurrence's result does not depend on
// where a sequence is cut, outputs and final state are those of the chunk size the caller named.
int tile_chunk(int chunk) { return chunk > 64 ? 64 : chunk; }

// The host-buffer forward overlaps its uploads, kernels and downloads: pieces of the batch go up on one internal
// stream, are computed on the caller's stream and come down on another internal stream, chained by events.  The two
// streams and the events are created once per device on first use and kept for the life of the process.
constexpr int kMaxPieces = 8;
constexpr int kMaxPipeDevices = 64;
struct HostPipe {
    bool ready = false;
    cudaStream_t up = nullptr, down = nullptr;
    cudaEvent_t start = nullptr, end = nullptr, uploaded[kMaxPieces] = {}, computed[kMaxPieces] = {};
};
std::mutex g_pipe_mutex;
HostPipe g_pipes[kMaxPipeDevices];

HostPipe *host_pipe()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxPipeDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe &hp = g_pipes[dev];
    if (!hp.ready) {
        bool ok = cudaStreamCreateWithFlags(&hp.up, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp.down, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.end, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < kMaxPieces; ++i)
            ok = cudaEventCreateWithFlags(&hp.uploaded[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.computed[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return nullptr;
        hp.ready = true;
    }
    return &hp;
}

// batch elements per piece and number of pieces of the host-buffer forward
void host_pieces(int B, int *per_piece, int *pieces)
{
    *per_piece = (B + kMaxPieces - 1) / kMaxPieces;
    *pieces = (B + *per_piece - 1) / *per_piece;
}

int validate_forward(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
                     const float *beta, const float *S0, void *o, void *o_im, float *S_T, int B, int T, int H,
                     int d_k, int d_v, int chunk, int dtype)
{
    if (!q || !k || !v || !alpha || !theta || !beta || !o) return SFDA_ERR_NULL;
    if (B < 1 || T < 1 || H < 1) return SFDA_ERR_SHAPE;
    const int rc = check_dims(d_k, d_v, chunk, dtype);
    if (rc != SFDA_OK) return rc;
    const void *ptrs[] = {q, k, v, alpha, theta, beta, S0, o, o_im, S_T};
    for (const void *p : ptrs)
        if (p && !aligned16(p)) return SFDA_ERR_ALIGN;
    return SFDA_OK;
}

sfda::ForwardArgs pack(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
                       const float *beta, const float *S0, void *o, void *o_im, float *S_T, int B, int T, int H,
                       int d_k, int d_v, int chunk, int dtype)
{
    sfda::ForwardArgs a;
    a.q = q; a.k = k; a.v = v; a.alpha = alpha; a.theta = theta; a.beta = beta; a.S0 = S0;
    a.o = o; a.o_im = o_im; a.S_T = S_T;
    a.B = B; a.T = T; a.H = H; a.d_k = d_k; a.d_v = d_v; a.chunk = tile_chunk(chunk); a.dtype = dtype;
    return a;
}

size_t round256(size_t x) { return (x + 255u) & ~(size_t)255u; }

// the stable parameterisation's scalars: 0 <= alpha_min <= alpha_max <= 1, theta_max and eps finite and >= 0
// (comparisons written so that a NaN fails them)
int check_param_scalars(float alpha_min, float alpha_max, float theta_max, float eps)
{
    const bool ok = alpha_min >= 0.f && alpha_min <= alpha_max && alpha_max <= 1.f && theta_max >= 0.f &&
                    theta_max <= 3.0e38f && eps >= 0.f && eps <= 3.0e38f;
    return ok ? SFDA_OK : SFDA_ERR_VALUE;
}

// workspace of sfda_forward_fused on the CUDA-core shapes: alpha, theta, beta and the normalised key
size_t staged_frontend_bytes(size_t rows, int d_k, int dtype)
{
    return 2 * round256(rows * (d_k / 2) * 4) + round256(rows * 4) + round256(rows * d_k * elem_bytes(dtype));
}

// Time slices of the two-level scan when the caller leaves the choice to the library: the largest power of two that
// keeps B H n within the SM count of the current device with at least 16 chunks per slice; 1 (do not slice) unless
// that is at least 4.
int auto_slices(int B, int T, int H, int chunk)
{
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return 1;
    int n = 1;
    while ((long long)2 * n * B * H <= n_sm && T % (2 * n * chunk) == 0 && T / (2 * n * chunk) >= 16) n *= 2;
    // One more doubling puts more slices than SMs on the machine; the chunk forward then cuts them into time slices
    // of its own and fills the SMs that n slices left idle.  Taken when its schedule is at least 8 % shorter (the
    // scan and the correction grow a little with n): 128 slices of 256 chunks -> 256 of 128 measured 4.00 -> 3.81 ms.
    if (n >= 4 && T % (2 * n * chunk) == 0 && T / (2 * n * chunk) >= 16) {
        int q = 1, bal = 0;
        double now = 0.0, then = 0.0;
        sfda::forward_ws_partition(n * B * H, T / (n * chunk), n_sm, true, &q, &bal, &now);
        sfda::forward_ws_partition(2 * n * B * H, T / (2 * n * chunk), n_sm, true, &q, &bal, &then);
        if (then < 0.92 * now) n *= 2;
    }
    return n >= 4 ? n : 1;      // three passes of T / n tokens each: fewer than four slices cannot pay
}

int step_common(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
                const float *beta, float *S, void *o, void *o_im, int B, int H, int d_k, int d_v, int dtype,
                const sfda::StepParam &par, void *stream)
{
    g_last_launches = 0;
    if (!q || !k || !v || !alpha || !theta || !beta || !S || !o) return SFDA_ERR_NULL;
    if (B < 1 || H < 1) return SFDA_ERR_SHAPE;
    const int rc = check_dims(d_k, d_v, 64, dtype);
    if (rc != SFDA_OK) return rc;
    const void *ptrs[] = {q, k, v, alpha, theta, beta, S, o, o_im};
    for (const void *p : ptrs)
        if (p && !aligned16(p)) return SFDA_ERR_ALIGN;
    sfda::StepArgs a;
    a.q = q; a.k = k; a.v = v; a.alpha = alpha; a.theta = theta; a.beta = beta;
    a.S = S; a.o = o; a.o_im = o_im;
    a.B = B; a.H = H; a.d_k = d_k; a.d_v = d_v; a.dtype = dtype;
    a.par = par;
    return sfda::launch_step(a, static_cast<cudaStream_t>(stream), &g_last_launches) == cudaSuccess ? SFDA_OK
                                                                                                    : SFDA_ERR_CUDA;
}

}  // namespace

extern "C" {

const char *sfda_status_string(int status)
{
    switch (status) {
        case SFDA_OK: return "ok";
        case SFDA_ERR_NULL: return "a required pointer is NULL";
        case SFDA_ERR_SHAPE: return "invalid shape (B, T, H >= 1; d_k even; chunk >= 1)";
        case SFDA_ERR_UNSUPPORTED: return "unsupported d_k / d_v / chunk / dtype";
        case SFDA_ERR_ALIGN: return "a pointer is not 16-byte aligned";
        case SFDA_ERR_WORKSPACE: return "workspace missing or too small";
        case SFDA_ERR_CUDA: return "CUDA runtime error at launch";
        case SFDA_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case SFDA_ERR_VALUE: return "a scalar of the stable parameterisation is out of range";
        default: return "unknown status";
    }
}

int sfda_plan(int T, int chunk, int *n_chunks, int *tail_len)
{
    if (!n_chunks || !tail_len) return SFDA_ERR_NULL;
    if (T < 1 || chunk < 1) return SFDA_ERR_SHAPE;
    const int nc = (T + chunk - 1) / chunk;
    *n_chunks = nc;
    *tail_len = T - (nc - 1) * chunk;
    return SFDA_OK;
}

size_t sfda_workspace_bytes(int B, int T, int H, int d_k, int d_v, int chunk, int dtype)
{
    if (B < 1 || T < 1 || H < 1 || check_dims(d_k, d_v, chunk, dtype) != SFDA_OK) return 0;
    sfda::ForwardArgs a{};
    a.B = B; a.T = T; a.H = H; a.d_k = d_k; a.d_v = d_v; a.chunk = tile_chunk(chunk); a.dtype = dtype;
    // the tensor-core path keeps a status word there, and the boundary states of its time slices
    return sfda::forward_ws_supported(a) ? sfda::forward_ws_scratch_bytes(B, H) : 0;
}

int sfda_forward_partition(int B, int T, int H, int d_k, int d_v, int chunk, int dtype, size_t workspace_bytes,
                           int n_sm, int *slices, int *balanced, int *ctas)
{
    if (!slices || !balanced || !ctas) return SFDA_ERR_NULL;
    if (B < 1 || T < 1 || H < 1 || n_sm < 1) return SFDA_ERR_SHAPE;
    const int rc = check_dims(d_k, d_v, chunk, dtype);
    if (rc != SFDA_OK) return rc;
    *slices = 1;
    *balanced = 0;
    *ctas = 0;
    sfda::ForwardArgs a{};
    a.B = B; a.T = T; a.H = H; a.d_k = d_k; a.d_v = d_v; a.chunk = tile_chunk(chunk); a.dtype = dtype;
    if (!sfda::forward_ws_supported(a) || workspace_bytes < 256) return SFDA_OK;
    const int BH = B * H, NC = (T + a.chunk - 1) / a.chunk;
    sfda::forward_ws_partition(BH, NC, n_sm, workspace_bytes >= sfda::forward_ws_scratch_bytes(B, H), slices, balanced, nullptr);
    const long long units = (long long)BH * *slices;
    *ctas = (int)(units < n_sm ? units : n_sm);
    return SFDA_OK;
}

int sfda_forward_simt(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
                      const float *beta, const float *S0, void *o, void *o_im, float *S_T, int B, int T, int H,
                      int d_k, int d_v, int chunk, int dtype, void *stream)
{
    g_last_launches = 0;
    const int rc = validate_forward(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    if (rc != SFDA_OK) return rc;
    const sfda::ForwardArgs a = pack(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    return sfda::launch_forward_simt(a, static_cast<cudaStream_t>(stream), &g_last_launches) == cudaSuccess
               ? SFDA_OK
               : SFDA_ERR_CUDA;
}

int sfda_forward(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
                 const float *beta, const float *S0, void *o, void *o_im, float *S_T, int B, int T, int H, int d_k,
                 int d_v, int chunk, int dtype, void *workspace, size_t workspace_bytes, void *stream)
{
    g_last_launches = 0;
    const int rc = validate_forward(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    if (rc != SFDA_OK) return rc;
    const sfda::ForwardArgs a = pack(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    // the tensor-core path runs with as little as its status block; the full size enables time slicing
    const size_t need = sfda::forward_ws_supported(a) ? sfda::kWsMinScratchBytes : 0;
    if (need > 0 && (!workspace || workspace_bytes < need)) return SFDA_ERR_WORKSPACE;
    if (workspace && !aligned16(workspace)) return SFDA_ERR_ALIGN;
    const cudaError_t e =
        sfda::forward_ws_supported(a)
            ? sfda::launch_forward_ws(a, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                                      &g_last_launches)
            : sfda::launch_forward_simt(a, static_cast<cudaStream_t>(stream), &g_last_launches);
    return e == cudaSuccess ? SFDA_OK : SFDA_ERR_CUDA;
}

int sfda_forward_phase(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
                       const float *beta, const float *S0, void *o, void *o_im, float *S_T, uint32_t *phase_turns,
                       int B, int T, int H, int d_k, int d_v, int chunk, int dtype, void *workspace,
                       size_t workspace_bytes, void *stream)
{
    g_last_launches = 0;
    const int rc = validate_forward(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    if (rc != SFDA_OK) return rc;
    if (!phase_turns) return SFDA_ERR_NULL;
    if (!aligned16(phase_turns)) return SFDA_ERR_ALIGN;
    if (chunk > 64) return SFDA_ERR_UNSUPPORTED;                         // one phase per 64-token tile is what is exported
    sfda::ForwardArgs a = pack(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    if (!sfda::forward_ws_supported(a)) return SFDA_ERR_UNSUPPORTED;     // the export belongs to the tensor-core kernel
    if (!workspace || workspace_bytes < sfda::kWsMinScratchBytes) return SFDA_ERR_WORKSPACE;
    if (!aligned16(workspace)) return SFDA_ERR_ALIGN;
    a.phase_turns = phase_turns;
    return sfda::launch_forward_ws(a, workspace, workspace_bytes, static_cast<cudaStream_t>(stream), &g_last_launches) ==
                   cudaSuccess
               ? SFDA_OK
               : SFDA_ERR_CUDA;
}

int sfda_forward_withheld_handoff(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
                                  const float *beta, const float *S0, void *o, void *o_im, float *S_T, int B, int T,
                                  int H, int d_k, int d_v, int chunk, int dtype, int slices, unsigned wait_ticks,
                                  void *workspace, size_t workspace_bytes, void *stream)
{
    g_last_launches = 0;
    const int rc = validate_forward(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    if (rc != SFDA_OK) return rc;
    sfda::ForwardArgs a = pack(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    if (!sfda::forward_ws_supported(a)) return SFDA_ERR_UNSUPPORTED;
    // at least two slices (so that something waits), a limit between 2^16 and 2^26 ticks (a few dozen microseconds to a
    // few dozen milliseconds), whole chunks per slice, and the full workspace (the hand-off buffers live there)
    if (slices < 2 || slices > 8 || wait_ticks < (1u << 16) || wait_ticks > (1u << 26)) return SFDA_ERR_VALUE;
    if (((T + a.chunk - 1) / a.chunk) % slices != 0) return SFDA_ERR_SHAPE;
    if (!workspace || workspace_bytes < sfda::forward_ws_scratch_bytes(B, H)) return SFDA_ERR_WORKSPACE;
    if (!aligned16(workspace)) return SFDA_ERR_ALIGN;
    a.debug_slices = slices;
    a.debug_withhold = 1;
    a.wait_ticks = wait_ticks;
    return sfda::launch_forward_ws(a, workspace, workspace_bytes, static_cast<cudaStream_t>(stream), &g_last_launches) ==
                   cudaSuccess
               ? SFDA_OK
               : SFDA_ERR_CUDA;
}

size_t sfda_forward_two_level_workspace_bytes(int B, int T, int H, int d_k, int d_v, int chunk, int dtype,
                                              int n_slices)
{
    if (B < 1 || T < 1 || H < 1 || n_slices < 0 || check_dims(d_k, d_v, chunk, dtype) != SFDA_OK) return 0;
    sfda::ForwardArgs a{};
    a.B = B; a.T = T; a.H = H; a.d_k = d_k; a.d_v = d_v; a.chunk = tile_chunk(chunk); a.dtype = dtype;
    if (!sfda::forward_ws_supported(a)) return 0;
    const int n = n_slices ? n_slices : auto_slices(B, T, H, tile_chunk(chunk));
    if (n == 1) return sfda::forward_ws_scratch_bytes(B, H);
    return sfda::forward_two_level_supported(a, n) ? sfda::forward_two_level_bytes(a, n) : 0;
}

int sfda_forward_two_level(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
                           const float *beta, const float *S0, void *o, void *o_im, float *S_T, int B, int T, int H,
                           int d_k, int d_v, int chunk, int dtype, int n_slices, void *workspace,
                           size_t workspace_bytes, void *stream)
{
    g_last_launches = 0;
    const int rc = validate_forward(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    if (rc != SFDA_OK) return rc;
    if (n_slices < 0 || n_slices == 1) return SFDA_ERR_SHAPE;
    const sfda::ForwardArgs a = pack(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    if (!sfda::forward_ws_supported(a)) return SFDA_ERR_UNSUPPORTED;
    if (workspace && !aligned16(workspace)) return SFDA_ERR_ALIGN;
    const int n = n_slices ? n_slices : auto_slices(B, T, H, tile_chunk(chunk));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n == 1) {       // nothing to gain: the plain forward
        if (!workspace || workspace_bytes < sfda::kWsMinScratchBytes) return SFDA_ERR_WORKSPACE;
        return sfda::launch_forward_ws(a, workspace, workspace_bytes, s, &g_last_launches) == cudaSuccess ? SFDA_OK
                                                                                                          : SFDA_ERR_CUDA;
    }
    if (!sfda::forward_two_level_supported(a, n)) return SFDA_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < sfda::forward_two_level_bytes(a, n)) return SFDA_ERR_WORKSPACE;
    return sfda::launch_forward_two_level(a, n, workspace, s, &g_last_launches) == cudaSuccess ? SFDA_OK
                                                                                                : SFDA_ERR_CUDA;
}

int sfda_forward_noalloc(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
                         const float *beta, const float *S0, void *o, void *o_im, float *S_T, int B, int T, int H,
                         int d_k, int d_v, int chunk, int dtype, void *stream)
{
    g_last_launches = 0;
    const int rc = validate_forward(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    if (rc != SFDA_OK) return rc;
    const sfda::ForwardArgs a = pack(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    if (!sfda::forward_ws_supported(a)) return SFDA_ERR_UNSUPPORTED;     // only the kernel that uses scratch
    if (sfda::kWsMinScratchBytes > SFDA_STATIC_SCRATCH_BYTES) return SFDA_ERR_WORKSPACE;
    return sfda::launch_forward_ws_static(a, static_cast<cudaStream_t>(stream), &g_last_launches) == cudaSuccess
               ? SFDA_OK
               : SFDA_ERR_CUDA;
}

int sfda_noalloc_status(void *stream, uint32_t *detail)
{
    uint32_t word = 0;
    if (sfda::read_static_status(static_cast<cudaStream_t>(stream), &word) != cudaSuccess) return SFDA_ERR_CUDA;
    if (detail) *detail = word;
    return word == 0 ? SFDA_OK : SFDA_ERR_TIMEOUT;
}

int sfda_workspace_status(const void *workspace, void *stream, uint32_t *detail)
{
    if (!workspace) return SFDA_ERR_NULL;
    uint32_t word = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return SFDA_ERR_CUDA;
    if (detail) *detail = word;
    return word == 0 ? SFDA_OK : SFDA_ERR_TIMEOUT;
}

int sfda_chunk_factors(const void *k, const float *alpha, const float *theta, const float *beta, float *Gamma,
                       float *Y, float *M, float *W, uint32_t *phase_turns, int B, int T, int H, int d_k, int chunk,
                       int dtype, void *stream)
{
    g_last_launches = 0;
    if (!k || !alpha || !theta || !beta) return SFDA_ERR_NULL;
    if (B < 1 || T < 1 || H < 1) return SFDA_ERR_SHAPE;
    const int rc = check_dims(d_k, 64, chunk, dtype);
    if (rc != SFDA_OK) return rc;
    // chunks of 128 and 256 tokens are composed of 64-token tiles, whose Gamma wait inside M: all four factor arrays are needed
    if (chunk > 64 && (!Gamma || !Y || !M || !W)) return SFDA_ERR_NULL;
    const void *ptrs[] = {k, alpha, theta, beta, Gamma, Y, M, W, phase_turns};
    for (const void *p : ptrs)
        if (p && !aligned16(p)) return SFDA_ERR_ALIGN;
    sfda::FactorArgs a;
    a.k = k; a.alpha = alpha; a.theta = theta; a.beta = beta;
    a.Gamma = Gamma; a.Y = Y; a.M = M; a.W = W; a.phase_turns = phase_turns;
    a.B = B; a.T = T; a.H = H; a.d_k = d_k; a.chunk = chunk; a.dtype = dtype;
    return sfda::launch_chunk_factors(a, static_cast<cudaStream_t>(stream), &g_last_launches) == cudaSuccess
               ? SFDA_OK
               : SFDA_ERR_CUDA;
}

int sfda_step(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
              const float *beta, float *S, void *o, void *o_im, int B, int H, int d_k, int d_v, int dtype,
              void *stream)
{
    return step_common(q, k, v, alpha, theta, beta, S, o, o_im, B, H, d_k, d_v, dtype, sfda::StepParam(), stream);
}

int sfda_forward_decoupled(const void *q, const void *k, const void *r, const void *v, const float *alpha,
                           const float *theta, const float *eta, const float *beta, const float *S0, void *o,
                           void *o_im, float *S_T, int B, int T, int H, int d_k, int d_v, int dtype, void *stream)
{
    g_last_launches = 0;
    if (!r || !eta) return SFDA_ERR_NULL;
    const int rc = validate_forward(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, 64, dtype);
    if (rc != SFDA_OK) return rc;
    if (!aligned16(r) || !aligned16(eta)) return SFDA_ERR_ALIGN;
    sfda::DecoupledArgs a;
    a.q = q; a.k = k; a.r = r; a.v = v; a.alpha = alpha; a.theta = theta; a.eta = eta; a.beta = beta; a.S0 = S0;
    a.o = o; a.o_im = o_im; a.S_T = S_T;
    a.B = B; a.T = T; a.H = H; a.d_k = d_k; a.d_v = d_v; a.dtype = dtype;
    return sfda::launch_forward_decoupled(a, static_cast<cudaStream_t>(stream), &g_last_launches) == cudaSuccess
               ? SFDA_OK
               : SFDA_ERR_CUDA;
}

int sfda_step_decoupled(const void *q, const void *k, const void *r, const void *v, const float *alpha,
                        const float *theta, const float *eta, const float *beta, float *S, void *o, void *o_im, int B,
                        int H, int d_k, int d_v, int dtype, void *stream)
{
    g_last_launches = 0;
    if (!r || !eta) return SFDA_ERR_NULL;
    if (!aligned16(r) || !aligned16(eta)) return SFDA_ERR_ALIGN;
    sfda::StepParam par;
    par.r = r;
    par.eta = eta;
    return step_common(q, k, v, alpha, theta, beta, S, o, o_im, B, H, d_k, d_v, dtype, par, stream);
}

int sfda_forward_blocks(const void *q, const void *k, const void *r, const void *v, const float *alpha,
                        const float *theta, const uint8_t *flip, const float *eta, const float *beta, const float *S0,
                        void *o, void *o_im, float *S_T, int B, int T, int H, int d_k, int d_v, int dtype, int erase,
                        void *stream)
{
    g_last_launches = 0;
    if (!r || !eta) return SFDA_ERR_NULL;
    const int rc = validate_forward(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, B, T, H, d_k, d_v, 64, dtype);
    if (rc != SFDA_OK) return rc;
    if (erase != SFDA_ERASE_COMPLEX && erase != SFDA_ERASE_REAL) return SFDA_ERR_VALUE;
    if (!aligned16(r) || !aligned16(eta) || (flip && !aligned16(flip))) return SFDA_ERR_ALIGN;
    sfda::DecoupledArgs a;
    a.q = q; a.k = k; a.r = r; a.v = v; a.alpha = alpha; a.theta = theta; a.eta = eta; a.beta = beta; a.S0 = S0;
    a.o = o; a.o_im = o_im; a.S_T = S_T;
    a.B = B; a.T = T; a.H = H; a.d_k = d_k; a.d_v = d_v; a.dtype = dtype;
    a.blocks = 1; a.real_erase = erase == SFDA_ERASE_REAL; a.flip = flip;
    return sfda::launch_forward_decoupled(a, static_cast<cudaStream_t>(stream), &g_last_launches) == cudaSuccess
               ? SFDA_OK
               : SFDA_ERR_CUDA;
}

int sfda_step_blocks(const void *q, const void *k, const void *r, const void *v, const float *alpha,
                     const float *theta, const uint8_t *flip, const float *eta, const float *beta, float *S, void *o,
                     void *o_im, int B, int H, int d_k, int d_v, int dtype, int erase, void *stream)
{
    g_last_launches = 0;
    if (!r || !eta) return SFDA_ERR_NULL;
    if (erase != SFDA_ERASE_COMPLEX && erase != SFDA_ERASE_REAL) return SFDA_ERR_VALUE;
    if (!aligned16(r) || !aligned16(eta) || (flip && !aligned16(flip))) return SFDA_ERR_ALIGN;
    sfda::StepParam par;
    par.r = r;
    par.eta = eta;
    par.blocks = 1; par.real_erase = erase == SFDA_ERASE_REAL; par.flip = flip;
    return step_common(q, k, v, alpha, theta, beta, S, o, o_im, B, H, d_k, d_v, dtype, par, stream);
}

int sfda_step_fused(const void *q, const void *k_raw, const void *v, const float *a_raw, const float *b_raw,
                    const float *c_raw, float alpha_min, float alpha_max, float theta_max, float eps, float *S,
                    void *o, void *o_im, int B, int H, int d_k, int d_v, int dtype, void *stream)
{
    g_last_launches = 0;
    const int rc = check_param_scalars(alpha_min, alpha_max, theta_max, eps);
    if (rc != SFDA_OK) return rc;
    sfda::StepParam par;
    par.fused = 1;
    par.a_lo = alpha_min; par.a_range = alpha_max - alpha_min; par.th_max = theta_max; par.eps = eps;
    return step_common(q, k_raw, v, a_raw, b_raw, c_raw, S, o, o_im, B, H, d_k, d_v, dtype, par, stream);
}

size_t sfda_forward_host_arena_bytes(int B, int T, int H, int d_k, int d_v, int chunk, int dtype, int want_o_im,
                                     int have_S0, int want_S_T)
{
    if (B < 1 || T < 1 || H < 1 || check_dims(d_k, d_v, chunk, dtype) != SFDA_OK) return 0;
    const size_t n = (size_t)B * T * H, eb = elem_bytes(dtype), m = d_k / 2;
    size_t total = 0;
    total += 2 * round256(n * d_k * eb);                      // q, k
    total += round256(n * d_v * eb);                          // v
    total += 2 * round256(n * m * 4);                         // alpha, theta
    total += (want_o_im ? 2 : 1) * round256(n * d_v * eb);    // o, o_im
    if (have_S0 || want_S_T) total += round256((size_t)B * H * d_k * d_v * 4);
    int per = 1, pieces = 1;
    host_pieces(B, &per, &pieces);
    // beta has 4 bytes per (token, head): a piece's share of one contiguous array would start on a 16-byte boundary
    // only when per * T * H is a multiple of four, so every piece gets a region of its own
    total += (size_t)pieces * round256((size_t)per * T * H * 4);
    total += (size_t)pieces * round256(sfda_workspace_bytes(per, T, H, d_k, d_v, chunk, dtype));   // one per piece
    return total;
}

int sfda_forward_host(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
                      const float *beta, const float *S0, void *o, void *o_im, float *S_T, int B, int T, int H,
                      int d_k, int d_v, int chunk, int dtype, void *arena, size_t arena_bytes, void *stream,
                      size_t *bytes_h2d, size_t *bytes_d2h)
{
    g_last_launches = 0;
    if (!q || !k || !v || !alpha || !theta || !beta || !o) return SFDA_ERR_NULL;
    if (B < 1 || T < 1 || H < 1) return SFDA_ERR_SHAPE;
    const int rc = check_dims(d_k, d_v, chunk, dtype);
    if (rc != SFDA_OK) return rc;
    const size_t need = sfda_forward_host_arena_bytes(B, T, H, d_k, d_v, chunk, dtype, o_im != nullptr,
                                                      S0 != nullptr, S_T != nullptr);
    if (!arena || arena_bytes < need) return SFDA_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(arena) & 255u) return SFDA_ERR_ALIGN;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    HostPipe *hp = host_pipe();
    if (!hp) return SFDA_ERR_CUDA;
    const size_t n = (size_t)B * T * H, eb = elem_bytes(dtype), m = d_k / 2;
    const size_t state_elems = (size_t)H * d_k * d_v;             // per batch element
    char *cur = static_cast<char *>(arena);
    auto take = [&](size_t bytes) { char *p = cur; cur += round256(bytes); return p; };
    char *dq = take(n * d_k * eb), *dk = take(n * d_k * eb), *dv = take(n * d_v * eb);
    char *da = take(n * m * 4), *dt = take(n * m * 4);
    char *dout = take(n * d_v * eb), *dout_im = o_im ? take(n * d_v * eb) : nullptr;
    char *dS = (S0 || S_T) ? take((size_t)B * state_elems * 4) : nullptr;
    int per = 1, pieces = 1;
    host_pieces(B, &per, &pieces);
    const size_t beta_stride = round256((size_t)per * T * H * 4);   // one 256-byte-aligned beta region per piece
    char *db = take((size_t)pieces * beta_stride);
    const size_t ws_bytes = sfda_workspace_bytes(per, T, H, d_k, d_v, chunk, dtype);
    char *ws0 = take((size_t)pieces * round256(ws_bytes));

    size_t h2d = 0, d2h = 0;
    bool ok = true;
    int launches = 0, status = SFDA_OK;
    auto copy = [&](void *dst, const void *src, size_t bytes, cudaMemcpyKind kind, cudaStream_t st) {
        ok = ok && cudaMemcpyAsync(dst, src, bytes, kind, st) == cudaSuccess;
        (kind == cudaMemcpyHostToDevice ? h2d : d2h) += bytes;
    };
    // everything enqueued on the caller's stream so far comes before the first copy of either direction
    ok = ok && cudaEventRecord(hp->start, s) == cudaSuccess && cudaStreamWaitEvent(hp->up, hp->start, 0) == cudaSuccess &&
         cudaStreamWaitEvent(hp->down, hp->start, 0) == cudaSuccess;
    for (int i = 0; ok && i < pieces; ++i) {
        const int b0 = i * per, nb = (b0 + per <= B ? per : B - b0);
        const size_t r0 = (size_t)b0 * T * H, rn = (size_t)nb * T * H;        // (token, head) rows of the piece
        const char *hq = static_cast<const char *>(q), *hk = static_cast<const char *>(k), *hv = static_cast<const char *>(v);
        copy(dq + r0 * d_k * eb, hq + r0 * d_k * eb, rn * d_k * eb, cudaMemcpyHostToDevice, hp->up);
        copy(dk + r0 * d_k * eb, hk + r0 * d_k * eb, rn * d_k * eb, cudaMemcpyHostToDevice, hp->up);
        copy(dv + r0 * d_v * eb, hv + r0 * d_v * eb, rn * d_v * eb, cudaMemcpyHostToDevice, hp->up);
        copy(da + r0 * m * 4, alpha + r0 * m, rn * m * 4, cudaMemcpyHostToDevice, hp->up);
        copy(dt + r0 * m * 4, theta + r0 * m, rn * m * 4, cudaMemcpyHostToDevice, hp->up);
        copy(db + (size_t)i * beta_stride, beta + r0, rn * 4, cudaMemcpyHostToDevice, hp->up);
        if (S0) copy(dS + b0 * state_elems * 4, S0 + b0 * state_elems, nb * state_elems * 4, cudaMemcpyHostToDevice, hp->up);
        ok = ok && cudaEventRecord(hp->uploaded[i], hp->up) == cudaSuccess &&
             cudaStreamWaitEvent(s, hp->uploaded[i], 0) == cudaSuccess;
        if (!ok) break;
        float *dSp = dS ? reinterpret_cast<float *>(dS) + b0 * state_elems : nullptr;
        const int frc = sfda_forward(dq + r0 * d_k * eb, dk + r0 * d_k * eb, dv + r0 * d_v * eb,
                                     reinterpret_cast<float *>(da) + r0 * m, reinterpret_cast<float *>(dt) + r0 * m,
                                     reinterpret_cast<float *>(db + (size_t)i * beta_stride), S0 ? dSp : nullptr, dout + r0 * d_v * eb,
                                     dout_im ? dout_im + r0 * d_v * eb : nullptr, S_T ? dSp : nullptr, nb, T, H, d_k, d_v,
                                     chunk, dtype, ws0 + (size_t)i * round256(ws_bytes), ws_bytes, stream);
        if (frc != SFDA_OK) {      // nothing of this piece was launched; what is already queued still has to be joined below
            status = frc;
            break;
        }
        launches += g_last_launches;
        ok = ok && cudaEventRecord(hp->computed[i], s) == cudaSuccess &&
             cudaStreamWaitEvent(hp->down, hp->computed[i], 0) == cudaSuccess;
        copy(static_cast<char *>(o) + r0 * d_v * eb, dout + r0 * d_v * eb, rn * d_v * eb, cudaMemcpyDeviceToHost, hp->down);
        if (o_im)
            copy(static_cast<char *>(o_im) + r0 * d_v * eb, dout_im + r0 * d_v * eb, rn * d_v * eb, cudaMemcpyDeviceToHost,
                 hp->down);
        if (S_T) copy(S_T + b0 * state_elems, dSp, nb * state_elems * 4, cudaMemcpyDeviceToHost, hp->down);
    }
    // The caller's stream is done when the last download is -- and, also after an error, only when every upload
    // already queued on the internal stream is: otherwise a reuse of the arena could race those copies.
    const bool joined = cudaEventRecord(hp->end, hp->down) == cudaSuccess && cudaStreamWaitEvent(s, hp->end, 0) == cudaSuccess &&
                        cudaEventRecord(hp->start, hp->up) == cudaSuccess && cudaStreamWaitEvent(s, hp->start, 0) == cudaSuccess;
    g_last_launches = launches;
    if (bytes_h2d) *bytes_h2d = h2d;
    if (bytes_d2h) *bytes_d2h = d2h;
    if (status != SFDA_OK) return status;
    return ok && joined ? SFDA_OK : SFDA_ERR_CUDA;
}

int sfda_frontend(const float *a_raw, const float *b_raw, const float *c_raw, const void *k_raw, float alpha_min,
                  float alpha_max, float theta_max, float eps, float *alpha, float *theta, float *beta, void *k,
                  int B, int T, int H, int d_k, int dtype, void *stream)
{
    g_last_launches = 0;
    if (!a_raw || !b_raw || !c_raw || !k_raw || !alpha || !theta || !beta || !k) return SFDA_ERR_NULL;
    if (B < 1 || T < 1 || H < 1) return SFDA_ERR_SHAPE;
    int rc = check_dims(d_k, 64, 64, dtype);
    if (rc != SFDA_OK) return rc;
    if ((rc = check_param_scalars(alpha_min, alpha_max, theta_max, eps)) != SFDA_OK) return rc;
    const void *ptrs[] = {a_raw, b_raw, c_raw, k_raw, alpha, theta, beta, k};
    for (const void *p : ptrs)
        if (!aligned16(p)) return SFDA_ERR_ALIGN;
    sfda::FrontendArgs f;
    f.a_raw = a_raw; f.b_raw = b_raw; f.c_raw = c_raw; f.k_raw = k_raw;
    f.alpha = alpha; f.theta = theta; f.beta = beta; f.k = k;
    f.rows = (long long)B * T * H; f.d_k = d_k; f.dtype = dtype;
    f.alpha_min = alpha_min; f.alpha_max = alpha_max; f.theta_max = theta_max; f.eps = eps;
    return sfda::launch_frontend(f, static_cast<cudaStream_t>(stream), &g_last_launches) == cudaSuccess ? SFDA_OK
                                                                                                         : SFDA_ERR_CUDA;
}

int sfda_frontend_backward(const float *a_raw, const float *b_raw, const float *c_raw, const void *k_raw,
                           float alpha_min, float alpha_max, float theta_max, float eps, const float *dalpha,
                           const float *dtheta, const float *dbeta, const void *dk, float *da, float *db, float *dc,
                           void *dk_raw, int B, int T, int H, int d_k, int dtype, void *stream)
{
    g_last_launches = 0;
    if (!a_raw || !b_raw || !c_raw || !k_raw || !dalpha || !dtheta || !dbeta || !dk || !da || !db || !dc || !dk_raw)
        return SFDA_ERR_NULL;
    if (B < 1 || T < 1 || H < 1) return SFDA_ERR_SHAPE;
    int rc = check_dims(d_k, 64, 64, dtype);
    if (rc != SFDA_OK) return rc;
    if ((rc = check_param_scalars(alpha_min, alpha_max, theta_max, eps)) != SFDA_OK) return rc;
    const void *ptrs[] = {a_raw, b_raw, c_raw, k_raw, dalpha, dtheta, dbeta, dk, da, db, dc, dk_raw};
    for (const void *p : ptrs)
        if (!aligned16(p)) return SFDA_ERR_ALIGN;
    sfda::FrontendArgs f;
    f.a_raw = a_raw; f.b_raw = b_raw; f.c_raw = c_raw; f.k_raw = k_raw;
    f.alpha = da; f.theta = db; f.beta = dc; f.k = dk_raw;
    f.rows = (long long)B * T * H; f.d_k = d_k; f.dtype = dtype;
    f.alpha_min = alpha_min; f.alpha_max = alpha_max; f.theta_max = theta_max; f.eps = eps;
    f.backward = 1; f.dalpha = dalpha; f.dtheta = dtheta; f.dbeta = dbeta; f.dk = dk;
    return sfda::launch_frontend(f, static_cast<cudaStream_t>(stream), &g_last_launches) == cudaSuccess ? SFDA_OK
                                                                                                         : SFDA_ERR_CUDA;
}

size_t sfda_forward_fused_workspace_bytes(int B, int T, int H, int d_k, int d_v, int chunk, int dtype)
{
    if (B < 1 || T < 1 || H < 1 || check_dims(d_k, d_v, chunk, dtype) != SFDA_OK) return 0;
    sfda::ForwardArgs a{};
    a.B = B; a.T = T; a.H = H; a.d_k = d_k; a.d_v = d_v; a.chunk = tile_chunk(chunk); a.dtype = dtype;
    if (sfda::forward_ws_supported(a)) return sfda::forward_ws_scratch_bytes(B, H);
    return staged_frontend_bytes((size_t)B * T * H, d_k, dtype);
}

int sfda_forward_fused(const void *q, const void *k_raw, const void *v, const float *a_raw, const float *b_raw,
                       const float *c_raw, float alpha_min, float alpha_max, float theta_max, float eps,
                       const float *S0, void *o, void *o_im, float *S_T, int B, int T, int H, int d_k, int d_v,
                       int chunk, int dtype, void *workspace, size_t workspace_bytes, void *stream)
{
    g_last_launches = 0;
    int rc = validate_forward(q, k_raw, v, a_raw, b_raw, c_raw, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    if (rc != SFDA_OK) return rc;
    if ((rc = check_param_scalars(alpha_min, alpha_max, theta_max, eps)) != SFDA_OK) return rc;
    if (workspace && !aligned16(workspace)) return SFDA_ERR_ALIGN;
    sfda::ForwardArgs a = pack(q, k_raw, v, a_raw, b_raw, c_raw, S0, o, o_im, S_T, B, T, H, d_k, d_v, chunk, dtype);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (sfda::forward_ws_supported(a)) {
        if (!workspace || workspace_bytes < sfda::kWsMinScratchBytes) return SFDA_ERR_WORKSPACE;
        a.fused = 1;
        a.alpha_min = alpha_min; a.alpha_max = alpha_max; a.theta_max = theta_max; a.eps = eps;
        return sfda::launch_forward_ws(a, workspace, workspace_bytes, s, &g_last_launches) == cudaSuccess ? SFDA_OK
                                                                                                          : SFDA_ERR_CUDA;
    }
    // other shapes: the parameterisation as a kernel of its own into the workspace, then the CUDA-core forward
    const size_t rows = (size_t)B * T * H;
    if (!workspace || workspace_bytes < staged_frontend_bytes(rows, d_k, dtype)) return SFDA_ERR_WORKSPACE;
    char *w = static_cast<char *>(workspace);
    sfda::FrontendArgs f;
    f.a_raw = a_raw; f.b_raw = b_raw; f.c_raw = c_raw; f.k_raw = k_raw;
    f.alpha = reinterpret_cast<float *>(w);
    f.theta = reinterpret_cast<float *>(w + round256(rows * (d_k / 2) * 4));
    f.beta = reinterpret_cast<float *>(w + 2 * round256(rows * (d_k / 2) * 4));
    f.k = w + 2 * round256(rows * (d_k / 2) * 4) + round256(rows * 4);
    f.rows = (long long)rows; f.d_k = d_k; f.dtype = dtype;
    f.alpha_min = alpha_min; f.alpha_max = alpha_max; f.theta_max = theta_max; f.eps = eps;
    if (sfda::launch_frontend(f, s, &g_last_launches) != cudaSuccess) return SFDA_ERR_CUDA;
    a.alpha = f.alpha; a.theta = f.theta; a.beta = f.beta; a.k = f.k;
    return sfda::launch_forward_simt(a, s, &g_last_launches) == cudaSuccess ? SFDA_OK : SFDA_ERR_CUDA;
}

size_t sfda_backward_workspace_bytes(int B, int T, int H, int d_k, int d_v, int dtype)
{
    if (B < 1 || T < 1 || H < 1 || check_dims(d_k, d_v, 64, dtype) != SFDA_OK) return 0;
    return sfda::backward_workspace_bytes(B, T, H, d_k, d_v);
}

int sfda_backward(const void *q, const void *k, const void *v, const float *alpha, const float *theta,
                  const float *beta, const float *S0, const void *d_o, const void *d_o_im, const float *dS_T,
                  void *dq, void *dk, void *dv, float *dalpha, float *dtheta, float *dbeta, float *dS0, int B, int T,
                  int H, int d_k, int d_v, int dtype, void *workspace, size_t workspace_bytes, void *stream)
{
    g_last_launches = 0;
    if (!q || !k || !v || !alpha || !theta || !beta || !d_o || !dq || !dk || !dv || !dalpha || !dtheta || !dbeta ||
        !dS0)
        return SFDA_ERR_NULL;
    if (B < 1 || T < 1 || H < 1) return SFDA_ERR_SHAPE;
    const int rc = check_dims(d_k, d_v, 64, dtype);
    if (rc != SFDA_OK) return rc;
    const void *ptrs[] = {q, k, v, alpha, theta, beta, S0, d_o, d_o_im, dS_T, dq, dk, dv, dalpha, dtheta, dbeta, dS0,
                          workspace};
    for (const void *p : ptrs)
        if (p && !aligned16(p)) return SFDA_ERR_ALIGN;
    if (!workspace || workspace_bytes < sfda::backward_workspace_bytes(B, T, H, d_k, d_v)) return SFDA_ERR_WORKSPACE;
    sfda::BackwardArgs a;
    a.q = q; a.k = k; a.v = v; a.d_o = d_o; a.d_o_im = d_o_im;
    a.alpha = alpha; a.theta = theta; a.beta = beta; a.S0 = S0; a.dS_T = dS_T;
    a.dq = dq; a.dk = dk; a.dv = dv; a.dalpha = dalpha; a.dtheta = dtheta; a.dbeta = dbeta; a.dS0 = dS0;
    a.B = B; a.T = T; a.H = H; a.d_k = d_k; a.d_v = d_v; a.dtype = dtype;
    return sfda::launch_backward(a, workspace, static_cast<cudaStream_t>(stream), &g_last_launches) == cudaSuccess
               ? SFDA_OK
               : SFDA_ERR_CUDA;
}

int sfda_last_launch_count(void) { return g_last_launches; }

}  // extern "C"
