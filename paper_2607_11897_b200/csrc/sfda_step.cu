// sfda_step: one-token recurrent decode (Section 3, Eq. "sfda" and o_t = S_t^* q_t).
//
// HBM-bound: per (batch, head) the d_k x d_v fp32 state is read once and written once; everything
// else is a few hundred bytes.  One CTA of 128 threads owns a block of kColTile value columns of one state (the
// columns of a state never interact: c = k^* S, the update and o = S^* q are all per column), so that a thread
// holds few enough registers for four or five CTAs per SM to overlap their loads, arithmetic and stores.
// A thread owns four adjacent
// columns (one 16-byte vector per row) of a group of complex rows, so every global access is a
// coalesced 128-bit load or store, and the whole slice a thread owns stays in registers between the
// two passes the update needs (first c = k^* (Lambda S), then S += k beta (v - c) and o = S^* q).
#include "sfda_common.cuh"
#include "sfda_internal.h"

namespace sfda {
namespace {

constexpr int kStepThreads = 128;
constexpr int kColTile = 64;   // value columns per CTA

template <int DK, int DV, typename T>
__global__ void __launch_bounds__(kStepThreads)
sfda_step_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
                 const float *__restrict__ alpha, const float *__restrict__ theta,
                 const float *__restrict__ beta, float *__restrict__ S, T *__restrict__ o,
                 T *__restrict__ o_im)
{
    constexpr int M = DK / 2;              // complex rows
    constexpr int CT = DV < kColTile ? DV : kColTile;   // columns of this CTA
    constexpr int CG = CT / 4;             // threads across one row (float4 each)
    constexpr int RG = kStepThreads / CG;  // row groups
    constexpr int R = M / RG;              // complex rows per thread
    static_assert(M % RG == 0, "row groups must divide the complex rows");

    __shared__ float s_lr[M], s_li[M], s_kr[M], s_ki[M], s_qr[M], s_qi[M];
    __shared__ float s_v[CT];
    __shared__ float s_red[RG][2][CT];

    const int tid = threadIdx.x;
    const size_t bh = blockIdx.x;
    const int c0 = blockIdx.y * CT;        // first column of this CTA
    const int cg = tid % CG, rg = tid / CG;

    float *Sbh = S + bh * (size_t)DK * DV + c0;

    // Issue the state loads first: they are the long-latency part.
    float4 sre[R], sim[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int j = rg * R + r;
        sre[r] = *reinterpret_cast<const float4 *>(Sbh + (size_t)(2 * j) * DV + 4 * cg);
        sim[r] = *reinterpret_cast<const float4 *>(Sbh + (size_t)(2 * j + 1) * DV + 4 * cg);
    }

    for (int j = tid; j < M; j += kStepThreads) {
        const float a = alpha[bh * M + j];
        float sn, cs;
        sincosf(theta[bh * M + j], &sn, &cs);
        s_lr[j] = a * cs;
        s_li[j] = a * sn;
        s_kr[j] = ld_val(k, bh * DK + 2 * j);
        s_ki[j] = ld_val(k, bh * DK + 2 * j + 1);
        s_qr[j] = ld_val(q, bh * DK + 2 * j);
        s_qi[j] = ld_val(q, bh * DK + 2 * j + 1);
    }
    for (int c = tid; c < CT; c += kStepThreads) s_v[c] = ld_val(v, bh * DV + c0 + c);
    const float bt = beta[bh];
    __syncthreads();

    // S <- Lambda S (2x2 rotation-decay per complex row);  partial c = k^* (Lambda S).
    float cre[4] = {0.f, 0.f, 0.f, 0.f}, cim[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int j = rg * R + r;
        const float lr = s_lr[j], li = s_li[j], kr = s_kr[j], ki = s_ki[j];
        float *pr = reinterpret_cast<float *>(&sre[r]);
        float *pi = reinterpret_cast<float *>(&sim[r]);
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const float nr = lr * pr[x] - li * pi[x];
            const float ni = lr * pi[x] + li * pr[x];
            pr[x] = nr;
            pi[x] = ni;
            cre[x] += kr * nr + ki * ni;   // conj(k) * s
            cim[x] += kr * ni - ki * nr;
        }
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        s_red[rg][0][4 * cg + x] = cre[x];
        s_red[rg][1][4 * cg + x] = cim[x];
    }
    __syncthreads();
    float ere[4], eim[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        float a = 0.f, b = 0.f;
#pragma unroll
        for (int g = 0; g < RG; ++g) {
            a += s_red[g][0][4 * cg + x];
            b += s_red[g][1][4 * cg + x];
        }
        ere[x] = bt * (s_v[4 * cg + x] - a);   // e = beta (v - c), v real
        eim[x] = -bt * b;
    }
    __syncthreads();   // s_red is reused below

    // S <- S + k e^T;  partial o = S^* q.
    float ore[4] = {0.f, 0.f, 0.f, 0.f}, oim[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int j = rg * R + r;
        const float kr = s_kr[j], ki = s_ki[j], qr = s_qr[j], qi = s_qi[j];
        float *pr = reinterpret_cast<float *>(&sre[r]);
        float *pi = reinterpret_cast<float *>(&sim[r]);
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const float nr = pr[x] + kr * ere[x] - ki * eim[x];
            const float ni = pi[x] + kr * eim[x] + ki * ere[x];
            pr[x] = nr;
            pi[x] = ni;
            ore[x] += nr * qr + ni * qi;   // conj(s) * q
            oim[x] += nr * qi - ni * qr;
        }
        *reinterpret_cast<float4 *>(Sbh + (size_t)(2 * j) * DV + 4 * cg) = sre[r];
        *reinterpret_cast<float4 *>(Sbh + (size_t)(2 * j + 1) * DV + 4 * cg) = sim[r];
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        s_red[rg][0][4 * cg + x] = ore[x];
        s_red[rg][1][4 * cg + x] = oim[x];
    }
    __syncthreads();
    for (int c = tid; c < CT; c += kStepThreads) {
        float a = 0.f, b = 0.f;
#pragma unroll
        for (int g = 0; g < RG; ++g) {
            a += s_red[g][0][c];
            b += s_red[g][1][c];
        }
        st_val(o, bh * DV + c0 + c, a);
        if (o_im) st_val(o_im, bh * DV + c0 + c, b);
    }
}

template <int DK, int DV, typename T>
cudaError_t launch_one(const StepArgs &a, cudaStream_t stream)
{
    const dim3 grid((unsigned)a.B * (unsigned)a.H, DV > kColTile ? DV / kColTile : 1);
    sfda_step_kernel<DK, DV, T><<<grid, kStepThreads, 0, stream>>>(
        static_cast<const T *>(a.q), static_cast<const T *>(a.k), static_cast<const T *>(a.v), a.alpha,
        a.theta, a.beta, a.S, static_cast<T *>(a.o), static_cast<T *>(a.o_im));
    return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch(const StepArgs &a, cudaStream_t stream)
{
    if (a.d_k == 128 && a.d_v == 128) return launch_one<128, 128, T>(a, stream);
    if (a.d_k == 128 && a.d_v == 64) return launch_one<128, 64, T>(a, stream);
    if (a.d_k == 64 && a.d_v == 128) return launch_one<64, 128, T>(a, stream);
    if (a.d_k == 64 && a.d_v == 64) return launch_one<64, 64, T>(a, stream);
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_step(const StepArgs &a, cudaStream_t stream, int *launches)
{
    const cudaError_t e = a.dtype == 1 ? dispatch<__nv_bfloat16>(a, stream) : dispatch<float>(a, stream);
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace sfda
