// Two-level scan over the time axis for few, long sequences.
//
// One sequence is one serial chain of chunks, so with fewer (batch, head) pairs than SMs most of the GPU idles.  The
// chunk transfer is affine in the state (Theorem "Exact affine chunk transfer"): over a time slice,
// S_out = P S_in + B with P (d_k/2 x d_k/2 complex) and B (the state the slice reaches from zero) independent of
// S_in.  So a sequence is cut into n slices that run as independent sequences:
//
//   pass 1a   every slice from a zero state (slice 0 from S_0): its B, and for slice 0 the final outputs;
//   pass 1b   every slice with v = 0 from the state [I | 0]: the first d_k/2 columns of what it reaches are P;
//   scan      S_1 = B_0,  S_{i+1} = P_i S_i + B_i   (n - 1 small complex products per pair, this file's kernel);
//   pass 2    every slice again from its true initial state: the outputs.
//
// [B][T] is contiguous, so slice i of batch element b is simply batch element b n + i of a [B n][T / n] problem on
// the same memory: the passes are plain calls of the chunk forward.  Three passes over the data, each n times as
// parallel: worth it when B H n fits the machine.  Exact up to the rounding of the forward itself (P and B carry its
// bf16 operand rounding once more).
#include "sfda_common.cuh"
#include "sfda_internal.h"

namespace sfda {
namespace {

constexpr int kScanThreads = 1024;

// S0 of pass 1b: the complex identity in the first M columns, zero elsewhere (paired rows: row 2j is Re of coordinate j).
__global__ void two_level_identity_kernel(float *__restrict__ S, int d_k, int d_v, size_t n_states)
{
    const size_t per = (size_t)d_k * d_v;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_states * per; i += (size_t)gridDim.x * blockDim.x) {
        const size_t e = i % per;
        const int row = (int)(e / d_v), col = (int)(e % d_v);
        S[i] = ((row & 1) == 0 && col == row / 2) ? 1.0f : 0.0f;
    }
}

// Pass 1a starts slice 0 from S_0 (or zero) and every other slice from zero.
__global__ void two_level_init_kernel(float *__restrict__ S, const float *__restrict__ S0, int n, int H, size_t per,
                                      size_t n_states)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_states * per; i += (size_t)gridDim.x * blockDim.x) {
        const size_t st = i / per, e = i % per;              // st = (b n + slice) H + h
        const size_t bq = st / H, h = st % H, b = bq / n, sl = bq % n;
        S[i] = (sl == 0 && S0) ? S0[(b * H + h) * per + e] : 0.0f;
    }
}

// One CTA per (batch, head) pair: S_1 = B_0 (slice 0 already started from S_0), S_{i+1} = P_i S_i + B_i; writes the
// initial state of every slice for pass 2 and the final state.  P_i: columns 0 .. M-1 of Pst, complex via paired rows.
template <int DK, int DV>
__global__ void __launch_bounds__(kScanThreads)
two_level_scan_kernel(const float *__restrict__ Bst, const float *__restrict__ Pst, const float *__restrict__ S0,
                      float *__restrict__ Sin, float *__restrict__ S_T, int n, int H)
{
    constexpr int M = DK / 2;
    extern __shared__ float sm[];
    float *Sr = sm, *Si = Sr + M * DV;             // current state (complex [M][DV])
    float *Pr = Si + M * DV, *Pi = Pr + M * (M + 1);   // P [M][M + 1]
    const int tid = threadIdx.x, bh = blockIdx.x, h = bh % H, b = bh / H;
    const size_t per = (size_t)DK * DV;
    auto state = [&](const float *base, int sl) { return base + (((size_t)b * n + sl) * H + h) * per; };

    // slice 0 starts from S_0
    float *dst0 = Sin + (((size_t)b * n) * H + h) * per;
    for (int i = tid; i < DK * DV; i += kScanThreads) dst0[i] = S0 ? S0[(size_t)bh * per + i] : 0.f;
    const float *B0 = state(Bst, 0);
    for (int i = tid; i < M * DV; i += kScanThreads) {
        const int j = i / DV, c = i % DV;
        Sr[i] = B0[(size_t)(2 * j) * DV + c];
        Si[i] = B0[(size_t)(2 * j + 1) * DV + c];
    }
    __syncthreads();
    for (int sl = 1; sl < n; ++sl) {
        float *dst = Sin + (((size_t)b * n + sl) * H + h) * per;
        for (int i = tid; i < M * DV; i += kScanThreads) {
            const int j = i / DV, c = i % DV;
            dst[(size_t)(2 * j) * DV + c] = Sr[i];
            dst[(size_t)(2 * j + 1) * DV + c] = Si[i];
        }
        const float *P = state(Pst, sl), *Bs = state(Bst, sl);
        for (int i = tid; i < M * M; i += kScanThreads) {
            const int j = i / M, l = i % M;
            Pr[j * (M + 1) + l] = P[(size_t)(2 * j) * DV + l];
            Pi[j * (M + 1) + l] = P[(size_t)(2 * j + 1) * DV + l];
        }
        __syncthreads();
        // thread = column c and a group of rows: next[j][c] = B[j][c] + sum_l P[j][l] S[l][c]
        constexpr int RG = kScanThreads / DV, RPT = M / RG;
        const int c = tid % DV, g = tid / DV;
        float nr[RPT], ni[RPT];
#pragma unroll
        for (int r = 0; r < RPT; ++r) {
            const int j = g + RG * r;
            nr[r] = Bs[(size_t)(2 * j) * DV + c];
            ni[r] = Bs[(size_t)(2 * j + 1) * DV + c];
        }
        for (int l = 0; l < M; ++l) {
            const float sr = Sr[l * DV + c], si = Si[l * DV + c];
#pragma unroll
            for (int r = 0; r < RPT; ++r) {
                const int j = g + RG * r;
                const float pr = Pr[j * (M + 1) + l], pi = Pi[j * (M + 1) + l];
                nr[r] += pr * sr - pi * si;
                ni[r] += pr * si + pi * sr;
            }
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < RPT; ++r) {
            const int j = g + RG * r;
            Sr[j * DV + c] = nr[r];
            Si[j * DV + c] = ni[r];
        }
        __syncthreads();
    }
    if (S_T) {
        for (int i = tid; i < M * DV; i += kScanThreads) {
            const int j = i / DV, c = i % DV;
            S_T[(size_t)bh * per + (size_t)(2 * j) * DV + c] = Sr[i];
            S_T[(size_t)bh * per + (size_t)(2 * j + 1) * DV + c] = Si[i];
        }
    }
}

size_t round256(size_t x) { return (x + 255u) & ~(size_t)255u; }

}  // namespace

bool forward_two_level_supported(const ForwardArgs &a, int n)
{
    ForwardArgs s = a;
    if (n < 2 || a.T % n != 0) return false;
    s.B = a.B * n;
    s.T = a.T / n;
    return s.T % a.chunk == 0 && forward_ws_supported(s) && a.d_v >= a.d_k / 2;
}

// Workspace: the chunk forward's own scratch for the [B n][T / n] problem, five sets of B n H states (initial states
// of pass 1a, B, [I | 0], P, initial states of pass 2), a zero v and an output nobody reads (pass 1b).
size_t forward_two_level_bytes(const ForwardArgs &a, int n)
{
    const size_t states = (size_t)a.B * n * a.H * a.d_k * a.d_v * 4;
    const size_t tokens = (size_t)a.B * a.T * a.H * a.d_v * 2;
    return round256(forward_ws_scratch_bytes(a.B * n, a.H)) + 5 * round256(states) + 2 * round256(tokens);
}

cudaError_t launch_forward_two_level(const ForwardArgs &a, int n, void *workspace, cudaStream_t stream, int *launches)
{
    const size_t n_states = (size_t)a.B * n * a.H, per = (size_t)a.d_k * a.d_v;
    const size_t states = round256(n_states * per * 4), tokens = round256((size_t)a.B * a.T * a.H * a.d_v * 2);
    const size_t fwd_bytes = forward_ws_scratch_bytes(a.B * n, a.H);
    char *w = static_cast<char *>(workspace);
    void *fwd_ws = w;                                   w += round256(fwd_bytes);
    float *S_a = reinterpret_cast<float *>(w);          w += states;
    float *B_st = reinterpret_cast<float *>(w);         w += states;
    float *S_id = reinterpret_cast<float *>(w);         w += states;
    float *P_st = reinterpret_cast<float *>(w);         w += states;
    float *S_in = reinterpret_cast<float *>(w);         w += states;
    void *v_zero = w;                                   w += tokens;
    void *o_dummy = w;

    cudaError_t e = cudaMemsetAsync(v_zero, 0, tokens, stream);
    if (e != cudaSuccess) return e;
    const unsigned fill_grid = (unsigned)((n_states * per + 255) / 256 < 4096 ? (n_states * per + 255) / 256 : 4096);
    two_level_init_kernel<<<fill_grid, 256, 0, stream>>>(S_a, a.S0, n, a.H, per, n_states);
    two_level_identity_kernel<<<fill_grid, 256, 0, stream>>>(S_id, a.d_k, a.d_v, n_states);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (launches) *launches += 2;

    ForwardArgs s = a;
    s.B = a.B * n;
    s.T = a.T / n;
    // pass 1a: B of every slice (slice 0 from S_0: its outputs are final, pass 2 recomputes them all the same)
    s.S0 = S_a; s.S_T = B_st;
    if ((e = launch_forward_ws(s, fwd_ws, fwd_bytes, stream, launches)) != cudaSuccess) return e;
    // pass 1b: P of every slice
    s.v = v_zero; s.S0 = S_id; s.S_T = P_st; s.o = o_dummy; s.o_im = nullptr;
    if ((e = launch_forward_ws(s, fwd_ws, fwd_bytes, stream, launches)) != cudaSuccess) return e;
    // scan over the slices
    const size_t smem = (size_t)(2 * (a.d_k / 2) * a.d_v + 2 * (a.d_k / 2) * (a.d_k / 2 + 1)) * 4;
    auto kern = two_level_scan_kernel<128, 128>;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    kern<<<(unsigned)(a.B * a.H), kScanThreads, smem, stream>>>(B_st, P_st, a.S0, S_in, a.S_T, n, a.H);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (launches) ++*launches;
    // pass 2: the outputs
    s.v = a.v; s.S0 = S_in; s.S_T = nullptr; s.o = a.o; s.o_im = a.o_im;
    return launch_forward_ws(s, fwd_ws, fwd_bytes, stream, launches);
}

}  // namespace sfda
