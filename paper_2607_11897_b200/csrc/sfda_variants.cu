// Forward of the write-decoupled variant (Section 3, paragraph "Write-decoupled variant", Eq. "sfda-decoupled-main"),
//
//     S_t = (I - eta_t k_t k_t^*) Lambda_t S_{t-1} + beta_t r_t v_t^*,        o_t = S_t^* q_t,
//
// token by token in fp32 on the CUDA cores: a reference path for the variant.  (The chunk-WY kernels of this
// library compute the tied model r = k, eta = beta; with a separate write direction a chunk needs a second
// rotated operand tile, two more Gram blocks and one more product.)  One CTA per (batch, head) pair and block of
// value columns -- the columns of a state never interact -- with the state in shared memory; the vectors of the next
// token are loaded into registers while the current one is worked on.
//
// The same kernel, instantiated with kBlk, runs the real-coordinate model with aligned 2 x 2 orthogonal control
// blocks (Eq. "intro-sfda-real"; Theorem "Dihedral phase-orientation memory" and the remark after it): a block is
// alpha R(theta) F^flip with F = diag(1, -1), i.e. the complex row is conjugated before it is multiplied by
// alpha e^{i theta}; and the erase term is either the complex k k^* or the real rank-one k k^T on R^{2m}, for which
// only the real part of k^* Z is taken.
#include "sfda_common.cuh"
#include "sfda_internal.h"

namespace sfda {
namespace {

constexpr int kVarThreads = 256;
constexpr int kVarCols = 32;      // value columns per CTA

template <int DK, typename T, bool kBlk>
__global__ void __launch_bounds__(kVarThreads)
sfda_forward_decoupled_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ r,
                              const T *__restrict__ v, const float *__restrict__ alpha, const float *__restrict__ theta,
                              const float *__restrict__ eta, const float *__restrict__ beta, const float *__restrict__ S0,
                              T *__restrict__ o, T *__restrict__ o_im, float *__restrict__ S_T, int T_, int H, int dv,
                              const uint8_t *__restrict__ flip, int real_erase)
{
    constexpr int M = DK / 2, CT = kVarCols, NG = kVarThreads / CT, RA = M / NG;   // row groups, rows per thread
    static_assert(M % NG == 0 && M + CT + 2 <= kVarThreads, "thread mappings");
    __shared__ float2 S[M][CT + 1];
    __shared__ float4 v_lk[M];        // (lam re, lam im, k re, k im)
    __shared__ float4 v_rq[M];        // (r re, r im, q re, q im)
    __shared__ float v_v[CT], red[NG][4][CT], scal[2];
    __shared__ float v_sg[kBlk ? M : 1];      // -1 where the block reflects (the row is conjugated first), else 1

    const int tid = threadIdx.x, c = tid % CT, g = tid / CT;
    const int bh = blockIdx.x, h = bh % H, b = bh / H, c0 = blockIdx.y * CT;
    for (int idx = tid; idx < M * CT; idx += kVarThreads) {
        const int j = idx / CT, cc = idx % CT;
        S[j][cc] = S0 ? make_float2(S0[((size_t)bh * DK + 2 * j) * dv + c0 + cc], S0[((size_t)bh * DK + 2 * j + 1) * dv + c0 + cc])
                      : make_float2(0.f, 0.f);
    }
    // token vectors, one token ahead: threads [0, M) take a coordinate (alpha, theta, k, r, q), the next CT a column
    // (v), two more eta and beta
    float r0 = 0.f, r1 = 0.f, r2 = 0.f, r3 = 0.f, r4 = 0.f, r5 = 0.f, r6 = 0.f, r7 = 0.f, r8 = 1.f;
    auto load_tok = [&](int t) {
        if (t >= T_) return;
        const size_t row = ((size_t)b * T_ + t) * H + h;
        if (tid < M) {
            r0 = alpha[row * M + tid];
            r1 = theta[row * M + tid];
            r2 = ld_val(k, row * DK + 2 * tid);
            r3 = ld_val(k, row * DK + 2 * tid + 1);
            r4 = ld_val(r, row * DK + 2 * tid);
            r5 = ld_val(r, row * DK + 2 * tid + 1);
            r6 = ld_val(q, row * DK + 2 * tid);
            r7 = ld_val(q, row * DK + 2 * tid + 1);
            if (kBlk && flip) r8 = flip[row * M + tid] ? -1.f : 1.f;
        } else if (tid < M + CT) {
            r0 = ld_val(v, row * dv + c0 + tid - M);
        } else if (tid == M + CT) {
            r0 = eta[row];
        } else if (tid == M + CT + 1) {
            r0 = beta[row];
        }
    };
    load_tok(0);
    __syncthreads();
    for (int t = 0; t < T_; ++t) {
        if (tid < M) {
            float sn, cs;
            sincosf(r1, &sn, &cs);
            v_lk[tid] = make_float4(r0 * cs, r0 * sn, r2, r3);
            v_rq[tid] = make_float4(r4, r5, r6, r7);
            if (kBlk) v_sg[tid] = r8;
        } else if (tid < M + CT) {
            v_v[tid - M] = r0;
        } else if (tid == M + CT) {
            scal[0] = r0;
        } else if (tid == M + CT + 1) {
            scal[1] = r0;
        }
        __syncthreads();
        load_tok(t + 1);
        // Z = Lambda S (kept in registers), partial c = k^* Z over this thread's rows
        float zr[RA], zi[RA], cr = 0.f, ci = 0.f;
#pragma unroll
        for (int x = 0; x < RA; ++x) {
            const int j = g + NG * x;
            const float4 lk = v_lk[j];
            float2 s = S[j][c];
            if (kBlk) s.y *= v_sg[j];
            zr[x] = lk.x * s.x - lk.y * s.y;
            zi[x] = lk.x * s.y + lk.y * s.x;
            cr += lk.z * zr[x] + lk.w * zi[x];
            ci += lk.z * zi[x] - lk.w * zr[x];
        }
        red[g][0][c] = cr;
        red[g][1][c] = ci;
        __syncthreads();
        float sr = 0.f, si = 0.f;
#pragma unroll
        for (int gg = 0; gg < NG; ++gg) {
            sr += red[gg][0][c];
            si += red[gg][1][c];
        }
        if (kBlk && real_erase) si = 0.f;                        // k k^T on R^{2m}: the real part of k^* Z only
        const float er = -scal[0] * sr, ei = -scal[0] * si;      // -eta c along k
        const float wv = scal[1] * v_v[c];                       //  beta v along r
        // S = Z + k e^T + r (beta v)^T;  partial o = S^* q
        float orr = 0.f, oi = 0.f;
#pragma unroll
        for (int x = 0; x < RA; ++x) {
            const int j = g + NG * x;
            const float4 lk = v_lk[j], rq = v_rq[j];
            const float nr = zr[x] + lk.z * er - lk.w * ei + rq.x * wv;
            const float ni = zi[x] + lk.z * ei + lk.w * er + rq.y * wv;
            S[j][c] = make_float2(nr, ni);
            orr += nr * rq.z + ni * rq.w;                         // conj(s) q
            oi += nr * rq.w - ni * rq.z;
        }
        red[g][2][c] = orr;
        red[g][3][c] = oi;
        __syncthreads();
        if (tid < CT) {
            float a = 0.f, bsum = 0.f;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) {
                a += red[gg][2][c];
                bsum += red[gg][3][c];
            }
            const size_t at = (((size_t)b * T_ + t) * H + h) * dv + c0 + c;
            st_val(o, at, a);
            if (o_im) st_val(o_im, at, bsum);
        }
        // (the next token's staging writes v_lk, v_rq, v_v, scal: every read of them happened before the barrier above;
        //  red[.][2..3] is read by the first warp while others may already write red[.][0..1] of the next token)
    }
    __syncthreads();
    if (S_T) {
        for (int idx = tid; idx < M * CT; idx += kVarThreads) {
            const int j = idx / CT, cc = idx % CT;
            S_T[((size_t)bh * DK + 2 * j) * dv + c0 + cc] = S[j][cc].x;
            S_T[((size_t)bh * DK + 2 * j + 1) * dv + c0 + cc] = S[j][cc].y;
        }
    }
}

template <int DK, typename T>
cudaError_t launch_typed(const DecoupledArgs &a, cudaStream_t stream)
{
    const dim3 grid((unsigned)(a.B * a.H), (unsigned)(a.d_v / kVarCols));
    if (a.blocks)
        sfda_forward_decoupled_kernel<DK, T, true><<<grid, kVarThreads, 0, stream>>>(
            static_cast<const T *>(a.q), static_cast<const T *>(a.k), static_cast<const T *>(a.r),
            static_cast<const T *>(a.v), a.alpha, a.theta, a.eta, a.beta, a.S0, static_cast<T *>(a.o),
            static_cast<T *>(a.o_im), a.S_T, a.T, a.H, a.d_v, a.flip, a.real_erase);
    else
        sfda_forward_decoupled_kernel<DK, T, false><<<grid, kVarThreads, 0, stream>>>(
            static_cast<const T *>(a.q), static_cast<const T *>(a.k), static_cast<const T *>(a.r),
            static_cast<const T *>(a.v), a.alpha, a.theta, a.eta, a.beta, a.S0, static_cast<T *>(a.o),
            static_cast<T *>(a.o_im), a.S_T, a.T, a.H, a.d_v, nullptr, 0);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_forward_decoupled(const DecoupledArgs &a, cudaStream_t stream, int *launches)
{
    cudaError_t e;
    if (a.dtype == 1)
        e = a.d_k == 128 ? launch_typed<128, __nv_bfloat16>(a, stream) : launch_typed<64, __nv_bfloat16>(a, stream);
    else
        e = a.d_k == 128 ? launch_typed<128, float>(a, stream) : launch_typed<64, float>(a, stream);
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace sfda
