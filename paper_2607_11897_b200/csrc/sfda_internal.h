// Host-side launcher prototypes shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace sfda {

struct ForwardArgs {
    const void *q, *k, *v;
    const float *alpha, *theta, *beta, *S0;
    void *o, *o_im;
    float *S_T;
    int B, T, H, d_k, d_v, chunk, dtype;
    // fused == 1 (tensor-core path only): alpha, theta, beta and k hold the raw inputs of the stable
    // parameterisation, which the kernel applies with these constants on the way in
    int fused = 0;
    float alpha_min = 0.f, alpha_max = 1.f, theta_max = 0.f, eps = 0.f;
    // tensor-core path, plain inputs only: [B][H][NC][m] chunk-closing integer phase, or nullptr
    uint32_t *phase_turns = nullptr;
    // tensor-core path, diagnostic launches: device-side wait limit in SM-clock ticks (0: the default of about a
    // second), a fixed number of time slices per sequence (0: the launcher's choice), and hand-offs between slices
    // that are written but never announced (every later slice then waits until the limit and gives up)
    uint32_t wait_ticks = 0;
    int debug_slices = 0, debug_withhold = 0;
};

struct FactorArgs {
    const void *k;
    const float *alpha, *theta, *beta;
    float *Gamma, *Y, *M, *W;
    uint32_t *phase_turns;
    int B, T, H, d_k, chunk, dtype;
};

// fused != 0: alpha, theta, beta, k hold the raw inputs of the stable parameterisation (decode kernel)
struct StepParam {
    int fused = 0;
    float a_lo = 0.f, a_range = 1.f, th_max = 0.f, eps = 0.f;
    // write-decoupled variant (r != nullptr): write direction r [B][H][d_k] in the dtype of q, erase strength eta [B][H]
    const void *r = nullptr;
    const float *eta = nullptr;
    // 2 x 2 orthogonal control blocks (blocks != 0, with r and eta): flip [B][H][m] bytes or nullptr (no reflections),
    // real_erase != 0: the erase term is the real rank-one k k^T on R^{2m} instead of the complex k k^*
    int blocks = 0, real_erase = 0;
    const uint8_t *flip = nullptr;
};

struct StepArgs {
    const void *q, *k, *v;
    const float *alpha, *theta, *beta;
    float *S;
    void *o, *o_im;
    int B, H, d_k, d_v, dtype;
    StepParam par;
};

struct FrontendArgs {
    const float *a_raw, *b_raw, *c_raw;
    const void *k_raw;
    float *alpha, *theta, *beta;
    void *k;
    long long rows;      // B * T * H
    int d_k, dtype;
    float alpha_min, alpha_max, theta_max, eps;
    // backward != 0: the derivative of the map; dalpha, dtheta, dbeta, dk are the incoming gradients and the four
    // output fields above receive da, db, dc, dk_raw
    int backward = 0;
    const float *dalpha = nullptr, *dtheta = nullptr, *dbeta = nullptr;
    const void *dk = nullptr;
};

struct BackwardArgs {
    const void *q, *k, *v, *d_o, *d_o_im;
    const float *alpha, *theta, *beta, *S0, *dS_T;
    void *dq, *dk, *dv;
    float *dalpha, *dtheta, *dbeta, *dS0;
    int B, T, H, d_k, d_v, dtype;
};

struct DecoupledArgs {
    const void *q, *k, *r, *v;
    const float *alpha, *theta, *eta, *beta, *S0;
    void *o, *o_im;
    float *S_T;
    int B, T, H, d_k, d_v, dtype;
    // 2 x 2 orthogonal control blocks: see StepParam; flip is [B][T][H][m] here
    int blocks = 0, real_erase = 0;
    const uint8_t *flip = nullptr;
};

// Each returns a cudaError_t from configuring / launching; *launches is incremented per kernel.
cudaError_t launch_forward_simt(const ForwardArgs &a, cudaStream_t stream, int *launches);
// Tensor-core path (bf16, d_k = d_v = 128, chunk = 64): warp-specialised, chunk-pipelined tcgen05 kernel.
// `status` is one device word the kernel sets when a bounded wait runs out; it is cleared on the stream
// before the launch.
bool forward_ws_supported(const ForwardArgs &a);
// `scratch` starts with that word (kWsMinScratchBytes suffice); with forward_ws_scratch_bytes(B, H) bytes the
// launcher may also cut every sequence into time slices that hand their boundary state over through the scratch.
constexpr size_t kWsMinScratchBytes = 256;
size_t forward_ws_scratch_bytes(int B, int H);
void forward_ws_partition(int BH, int NC, int n_sm, bool cuts_allowed, int *slices, int *balanced, double *periods);
// clear_status = false keeps what an earlier launch on the same scratch block left in the status word.
cudaError_t launch_forward_ws(const ForwardArgs &a, void *scratch, size_t scratch_bytes, cudaStream_t stream,
                              int *launches, bool clear_status = true);
// The same kernel on the library's own statically allocated scratch block (kStaticScratchBytes), and a read of
// the status word kept there (synchronises the stream).  Neither allocates.
constexpr size_t kStaticScratchBytes = 256;
cudaError_t launch_forward_ws_static(const ForwardArgs &a, cudaStream_t stream, int *launches);
cudaError_t read_static_status(cudaStream_t stream, uint32_t *word);
cudaError_t launch_chunk_factors(const FactorArgs &a, cudaStream_t stream, int *launches);
cudaError_t launch_step(const StepArgs &a, cudaStream_t stream, int *launches);
// Two-level scan over n time slices of every sequence (tensor-core shapes, T a multiple of n * chunk): three passes
// of the chunk forward on the [B n][T / n] view of the same memory plus a small scan kernel.
bool forward_two_level_supported(const ForwardArgs &a, int n);
size_t forward_two_level_bytes(const ForwardArgs &a, int n);
cudaError_t launch_forward_two_level(const ForwardArgs &a, int n, void *workspace, cudaStream_t stream, int *launches);
// Reverse-mode derivative, token by token in fp32 (every supported d_k, d_v and dtype); the workspace holds the
// checkpointed states.
size_t backward_workspace_bytes(int B, int T, int H, int d_k, int d_v);
cudaError_t launch_backward(const BackwardArgs &a, void *workspace, cudaStream_t stream, int *launches);
// Forward of the write-decoupled variant, token by token in fp32 (every supported d_k, d_v and dtype).
cudaError_t launch_forward_decoupled(const DecoupledArgs &a, cudaStream_t stream, int *launches);
// Stable parameterisation as a kernel of its own (every supported d_k and dtype).
cudaError_t launch_frontend(const FrontendArgs &a, cudaStream_t stream, int *launches);

}  // namespace sfda
