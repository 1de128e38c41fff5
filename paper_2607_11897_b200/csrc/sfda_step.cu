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

// 16-byte load of state that stays where it is written: the loads must be in flight before the (short) preamble
// runs, whatever else the preamble has to compute.
__device__ __forceinline__ float4 ld_state(const float *p)
{
    float4 v;
    asm volatile("ld.global.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
    return v;
}

// kMode: 0 the tied recurrence; 1 the same on raw inputs of the stable parameterisation; 2 the write-decoupled
// variant S_t = (I - eta k k^*) Lambda S_{t-1} + beta r v^* (Section 3, Eq. "sfda-decoupled-main"); 3 the same with
// 2 x 2 orthogonal control blocks alpha R(theta) F^flip (a reflecting block conjugates the complex row first) and
// the choice of the real rank-one erase k k^T on R^{2m} (Eq. "intro-sfda-real"), which takes Re(k^* Z) only.
template <int DK, int DV, typename T, int kMode>
__global__ void __launch_bounds__(kStepThreads)
sfda_step_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
                 const float *__restrict__ alpha, const float *__restrict__ theta,
                 const float *__restrict__ beta, float *__restrict__ S, T *__restrict__ o,
                 T *__restrict__ o_im, const StepParam par)
{
    constexpr bool kFused = kMode == 1, kDec = kMode >= 2, kBlk = kMode == 3;
    constexpr int M = DK / 2;              // complex rows
    constexpr int CT = DV < kColTile ? DV : kColTile;   // columns of this CTA
    constexpr int CG = CT / 4;             // threads across one row (float4 each)
    constexpr int RG = kStepThreads / CG;  // row groups
    constexpr int R = M / RG;              // complex rows per thread
    static_assert(M % RG == 0, "row groups must divide the complex rows");

    __shared__ float s_lr[M], s_li[M], s_kr[M], s_ki[M], s_qr[M], s_qi[M];
    __shared__ float s_v[CT];
    __shared__ float s_red[RG][2][CT];
    __shared__ float s_norm[kStepThreads / 32];
    __shared__ float s_rr[kDec ? M : 1], s_ri[kDec ? M : 1];      // write direction r of the decoupled variant
    __shared__ float s_sg[kBlk ? M : 1];                          // -1 where the block reflects, else 1

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
        sre[r] = ld_state(Sbh + (size_t)(2 * j) * DV + 4 * cg);
        sim[r] = ld_state(Sbh + (size_t)(2 * j + 1) * DV + 4 * cg);
    }

    // kFused: alpha, theta, beta, k arrive raw and go through the stable parameterisation of Section 3 first
    // (Eqs. "param-alpha", "param-theta", "param-beta", "param-key"); a few hundred values per state, nothing
    // beside the 128 KB of state traffic.
    // Every global load of the preamble is issued before anything waits for one of them.
    static_assert(M <= kStepThreads && CT <= kStepThreads, "one coordinate and one column per thread at most");
    float a = 1.f, th = 0.f, kr0 = 0.f, ki0 = 0.f, qr0 = 0.f, qi0 = 0.f, v0 = 0.f, rr0 = 0.f, ri0 = 0.f;
    const float eta = kDec ? par.eta[bh] : 0.f;
    float sg0 = 1.f;
    if (kDec && tid < M) {
        rr0 = ld_val(static_cast<const T *>(par.r), bh * DK + 2 * tid);
        ri0 = ld_val(static_cast<const T *>(par.r), bh * DK + 2 * tid + 1);
        if (kBlk && par.flip) sg0 = par.flip[bh * M + tid] ? -1.f : 1.f;
    }
    if (tid < M) {
        a = alpha[bh * M + tid];
        th = theta[bh * M + tid];
        kr0 = ld_val(k, bh * DK + 2 * tid);
        ki0 = ld_val(k, bh * DK + 2 * tid + 1);
        qr0 = ld_val(q, bh * DK + 2 * tid);
        qi0 = ld_val(q, bh * DK + 2 * tid + 1);
    }
    if (tid < CT) v0 = ld_val(v, bh * DV + c0 + tid);
    float bt = beta[bh];
    float ss = 0.f;                        // this thread's share of |k_raw|^2
    if (tid < M) {
        if (kFused) {
            // sigmoid(x) = 1 / (1 + e^-x), tanh(x) = 1 - 2 / (1 + e^2x) with the fast exponential and division
            // (absolute error about 1e-7; both saturate correctly through infinity and zero)
            a = fmaf(par.a_range, __fdividef(1.0f, 1.0f + __expf(-a)), par.a_lo);
            th = fmaf(-2.0f * par.th_max, __fdividef(1.0f, 1.0f + __expf(2.0f * th)), par.th_max);
            ss = fmaf(kr0, kr0, ki0 * ki0);
        }
        float sn, cs;
        sincosf(th, &sn, &cs);
        s_lr[tid] = a * cs;
        s_li[tid] = a * sn;
        s_kr[tid] = kr0;
        s_ki[tid] = ki0;
        s_qr[tid] = qr0;
        s_qi[tid] = qi0;
        if (kDec) {
            s_rr[tid] = rr0;
            s_ri[tid] = ri0;
        }
        if (kBlk) s_sg[tid] = sg0;
    }
    if (tid < CT) s_v[tid] = v0;
    constexpr int kKeyWarps = (M + 31) / 32;       // the warps whose threads read key coordinates above
    if (kFused) {
        bt = __fdividef(1.0f, 1.0f + __expf(-bt));
        if (tid < 32 * kKeyWarps) {                // warp-uniform
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
            if ((tid & 31) == 0) s_norm[tid >> 5] = ss;
        }
    }
    __syncthreads();
    // s = 1 / (|k_raw| + eps).  The shared key stays raw: with k = s k_raw, c = s (k_raw^* Lambda S) and
    // S += k e^T = k_raw (s e)^T, so the scale enters twice per column instead of twice per state row.
    float sk = 1.0f;
    if (kFused) {
        float n2 = 0.f;
#pragma unroll
        for (int w = 0; w < kKeyWarps; ++w) n2 += s_norm[w];
        sk = __fdividef(1.0f, fmaxf(__fsqrt_rn(n2) + par.eps, 1.0e-30f));  // a zero key with eps = 0 stays zero
    }

    // S <- Lambda S (2x2 rotation-decay per complex row);  partial c = k^* (Lambda S).
    float cre[4] = {0.f, 0.f, 0.f, 0.f}, cim[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int j = rg * R + r;
        const float lr = s_lr[j], li = s_li[j], kr = s_kr[j], ki = s_ki[j];
        float *pr = reinterpret_cast<float *>(&sre[r]);
        float *pi = reinterpret_cast<float *>(&sim[r]);
        const float sg = kBlk ? s_sg[j] : 1.f;
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const float si = kBlk ? sg * pi[x] : pi[x];
            const float nr = lr * pr[x] - li * si;
            const float ni = lr * si + li * pr[x];
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
        if (kDec) {                            // erase part -eta c along k; the write beta v goes along r below
            ere[x] = -eta * a;
            eim[x] = kBlk && par.real_erase ? 0.f : -eta * b;
        } else if (kFused) {                   // c = s c_raw; e -> s e for the raw-key update
            ere[x] = sk * bt * (s_v[4 * cg + x] - sk * a);
            eim[x] = -sk * bt * sk * b;
        } else {
            ere[x] = bt * (s_v[4 * cg + x] - a);   // e = beta (v - c), v real
            eim[x] = -bt * b;
        }
    }
    __syncthreads();   // s_red is reused below

    // S <- S + k e^T;  partial o = S^* q.
    float ore[4] = {0.f, 0.f, 0.f, 0.f}, oim[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int j = rg * R + r;
        const float kr = s_kr[j], ki = s_ki[j], qr = s_qr[j], qi = s_qi[j];
        const float wr = kDec ? bt * s_rr[j] : 0.f, wi = kDec ? bt * s_ri[j] : 0.f;     // beta r
        float *pr = reinterpret_cast<float *>(&sre[r]);
        float *pi = reinterpret_cast<float *>(&sim[r]);
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            float nr = pr[x] + kr * ere[x] - ki * eim[x];
            float ni = pi[x] + kr * eim[x] + ki * ere[x];
            if (kDec) {                        // + beta r v^T (v real)
                nr = fmaf(wr, s_v[4 * cg + x], nr);
                ni = fmaf(wi, s_v[4 * cg + x], ni);
            }
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
    if (a.par.r && a.par.blocks)
        sfda_step_kernel<DK, DV, T, 3><<<grid, kStepThreads, 0, stream>>>(
            static_cast<const T *>(a.q), static_cast<const T *>(a.k), static_cast<const T *>(a.v), a.alpha,
            a.theta, a.beta, a.S, static_cast<T *>(a.o), static_cast<T *>(a.o_im), a.par);
    else if (a.par.r)
        sfda_step_kernel<DK, DV, T, 2><<<grid, kStepThreads, 0, stream>>>(
            static_cast<const T *>(a.q), static_cast<const T *>(a.k), static_cast<const T *>(a.v), a.alpha,
            a.theta, a.beta, a.S, static_cast<T *>(a.o), static_cast<T *>(a.o_im), a.par);
    else if (a.par.fused)
        sfda_step_kernel<DK, DV, T, 1><<<grid, kStepThreads, 0, stream>>>(
            static_cast<const T *>(a.q), static_cast<const T *>(a.k), static_cast<const T *>(a.v), a.alpha,
            a.theta, a.beta, a.S, static_cast<T *>(a.o), static_cast<T *>(a.o_im), a.par);
    else
        sfda_step_kernel<DK, DV, T, 0><<<grid, kStepThreads, 0, stream>>>(
            static_cast<const T *>(a.q), static_cast<const T *>(a.k), static_cast<const T *>(a.v), a.alpha,
            a.theta, a.beta, a.S, static_cast<T *>(a.o), static_cast<T *>(a.o_im), a.par);
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
