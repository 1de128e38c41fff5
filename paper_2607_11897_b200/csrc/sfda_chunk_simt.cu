// fp32 CUDA-core chunk-WY forward.
//
// What is computed per chunk (C tokens, one (batch, head) pair, gamma_t = prod_{s<=t} lambda_s inside
// the chunk, written gamma_t = a_t e^{i phi_t}):
//
//   k'_t = e^{-i phi_t} k_t,  q'_t = e^{-i phi_t} q_t            (rotated keys / queries)
//   Kt[t][i] = k_t^* diag(gamma_t/gamma_i) k_i = sum_j conj(k'_tj) k'_ij a_tj/a_ij      (i < t)
//   Aq[t][i] = q_t^* diag(gamma_t/gamma_i) k_i = sum_j conj(q'_tj) k'_ij a_tj/a_ij      (i <= t)
//   R = V - W^* S_0,  W_t = conj(gamma_t) k_t                      (W of Theorem "Constructive ... recursion")
//   (I + D_beta Kt) E = D_beta R                                   (the unit lower triangular WY system;
//        rows e_t^T = beta_t (v_t^T - k_t^* Lambda_t S_{t-1}); this is M of Eq. "constructive-M" applied)
//   o_t^* = (conj(gamma_t) q_t)^* S_0 + sum_{i<=t} Aq[t][i] e_i^T   (Theorem "Prefix outputs inside a chunk")
//   S_C = Gamma_C S_0 + sum_t (gamma_C/gamma_t) k_t e_t^T          (Eq. "apply-transfer" with B = Y M V)
//
// Only ratios a_t/a_i <= 1 are ever formed, so any alpha in [0, 1] is safe here.
#include "sfda_common.cuh"
#include "sfda_internal.h"

namespace sfda {
namespace {

constexpr int kThreads = 256;
constexpr int kSlice = 32;  // value columns per CTA of the forward kernel

// Index of the pair (t, i), i <= t, in row-major order of the lower triangle.
__device__ __forceinline__ void tri_decode(int p, int *t, int *i)
{
    int r = (int)((sqrtf(8.f * (float)p + 1.f) - 1.f) * 0.5f);
    while ((r + 1) * (r + 2) / 2 <= p) ++r;
    while (r * (r + 1) / 2 > p) --r;
    *t = r;
    *i = p - r * (r + 1) / 2;
}

template <int DK, int C>
struct ChunkSmem {
    static constexpr int M = DK / 2;
    static constexpr int KS = DK + 2;  // row stride of kp / qp (floats): spreads rows over banks
    static constexpr int LS = M + 1;   // row stride of lg
    static constexpr int GS = C + 1;   // row stride of the Gram matrices
    float *kp, *qp, *lg, *gcr, *gci, *lgC, *beta, *scan;
    __device__ explicit ChunkSmem(float *base)
    {
        kp = base;
        qp = kp + C * KS;
        lg = qp + C * KS;
        gcr = lg + C * LS;
        gci = gcr + M;
        lgC = gci + M;
        beta = lgC + M;
        scan = beta + C;                                   // [2][kThreads]: group totals of the scan
    }
    static constexpr int floats = 2 * C * KS + C * LS + 3 * M + C + 2 * kThreads;
};

// Loads one chunk of k (and q when given), alpha, theta, beta; leaves in shared memory the rotated
// keys / queries, the cumulative log-decay lg[t][j] = sum_{s<=t} log alpha_sj, the closing phase
// e^{i phi_C} and lg_C.  Tokens past `len` are neutral (alpha = 1, theta = 0, beta = 0, k = q = 0).
// When turns_out is not NULL the chunk-local cumulative phase turns of real tokens are written there.
template <int DK, int C, typename T>
__device__ void load_and_rotate(const ChunkSmem<DK, C> &sm, const T *__restrict__ k, const T *__restrict__ q,
                                const float *__restrict__ alpha, const float *__restrict__ theta,
                                const float *__restrict__ beta, uint32_t *__restrict__ turns_out, int b,
                                int h, int T_, int H, int t0, int len)
{
    constexpr int M = DK / 2;
    using S = ChunkSmem<DK, C>;
    // thread = (coordinate j, group g of TG consecutive tokens): every global load of the thread is issued before the
    // first one is used; the prefix sums run inside a group first and the groups are chained through shared memory
    constexpr int G = kThreads / M, TG = C / G;
    static_assert(kThreads % M == 0 && C % G == 0, "the scan's groups must tile the chunk");
    const int tid = threadIdx.x;
    const int j = tid % M, g = tid / M;
    float lgv[TG], kr[TG], ki[TG], qr[TG], qi[TG];
    uint32_t tu[TG];
#pragma unroll
    for (int x = 0; x < TG; ++x) {
        const int t = g * TG + x;
        float al = 1.f, th = 0.f;
        kr[x] = ki[x] = qr[x] = qi[x] = 0.f;
        if (t < len) {
            const size_t row = ((size_t)b * T_ + t0 + t) * H + h;
            al = alpha[row * M + j];
            th = theta[row * M + j];
            kr[x] = ld_val(k, row * DK + 2 * j);
            ki[x] = ld_val(k, row * DK + 2 * j + 1);
            if (q) {
                qr[x] = ld_val(q, row * DK + 2 * j);
                qi[x] = ld_val(q, row * DK + 2 * j + 1);
            }
        }
        lgv[x] = al;
        tu[x] = __float_as_uint(th);
    }
    if (tid < C) sm.beta[tid] = tid < len ? beta[((size_t)b * T_ + t0 + tid) * H + h] : 0.f;
    float acc = 0.f;
    uint32_t ta = 0u;
#pragma unroll
    for (int x = 0; x < TG; ++x) {
        acc += log_decay(lgv[x]);
        ta += phase_to_turns(__uint_as_float(tu[x]));
        lgv[x] = acc;
        tu[x] = ta;
    }
    float *grp_lg = sm.scan;                                        // [G][M]
    uint32_t *grp_tu = reinterpret_cast<uint32_t *>(sm.scan + G * M);
    grp_lg[g * M + j] = acc;
    grp_tu[g * M + j] = ta;
    __syncthreads();
    float base = 0.f;
    uint32_t tb = 0u;
    for (int gg = 0; gg < g; ++gg) {
        base += grp_lg[gg * M + j];
        tb += grp_tu[gg * M + j];
    }
#pragma unroll
    for (int x = 0; x < TG; ++x) {
        const int t = g * TG + x;
        const float l = base + lgv[x];
        const uint32_t tt = tb + tu[x];
        if (turns_out && t < len) turns_out[(((size_t)b * T_ + t0 + t) * H + h) * M + j] = tt;
        float cs, sn;
        turns_to_cos_sin(tt, &cs, &sn);
        sm.lg[t * S::LS + j] = l;
        sm.kp[t * S::KS + 2 * j] = kr[x] * cs + ki[x] * sn;         // e^{-i phi} (kr + i ki)
        sm.kp[t * S::KS + 2 * j + 1] = ki[x] * cs - kr[x] * sn;
        sm.qp[t * S::KS + 2 * j] = qr[x] * cs + qi[x] * sn;
        sm.qp[t * S::KS + 2 * j + 1] = qi[x] * cs - qr[x] * sn;
        if (t == C - 1) {
            sm.gcr[j] = cs;
            sm.gci[j] = sn;
            sm.lgC[j] = l;
        }
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// forward
// ------------------------------------------------------------------------------------------------
template <int DK, int C>
constexpr int forward_smem_floats()
{
    return ChunkSmem<DK, C>::floats + 2 * (DK / 2) * kSlice  // state (re, im)
           + 4 * C * (C + 1)                                  // Kt, Aq (re, im)
           + 2 * C * kSlice                                   // E (re, im)
           + 2 * C * (DK / 2 + 1);                            // a_t and a_C / a_t of the chunk
}

template <int DK, int C, typename T>
__global__ void __launch_bounds__(kThreads)
sfda_forward_simt_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
                         const float *__restrict__ alpha, const float *__restrict__ theta,
                         const float *__restrict__ beta, const float *__restrict__ S0, T *__restrict__ o,
                         T *__restrict__ o_im, float *__restrict__ S_T, int T_, int H, int dv)
{
    constexpr int M = DK / 2;
    using SM = ChunkSmem<DK, C>;
    extern __shared__ __align__(16) float smem[];
    const SM sm(smem);
    float *Sre = smem + SM::floats;
    float *Sim = Sre + M * kSlice;
    float *Ktr = Sim + M * kSlice;
    float *Kti = Ktr + C * SM::GS;
    float *Aqr = Kti + C * SM::GS;
    float *Aqi = Aqr + C * SM::GS;
    float *Er = Aqi + C * SM::GS;
    float *Ei = Er + C * kSlice;
    float *aw = Ei + C * kSlice;          // [C][LS]  a_t = exp(lg_t)           (<= 1)
    float *yw = aw + C * SM::LS;          // [C][LS]  a_C / a_t = exp(lg_C - lg_t)  (<= 1)

    const int tid = threadIdx.x, lane = tid % 32, wid = tid / 32;
    const int nsl = dv / kSlice;
    const int slice = blockIdx.x % nsl;
    const int bh = blockIdx.x / nsl;
    const int h = bh % H, b = bh / H;
    const int c0 = slice * kSlice;

    for (int idx = tid; idx < M * kSlice; idx += kThreads) {
        const int j = idx / kSlice, c = idx % kSlice;
        Sre[idx] = S0 ? S0[((size_t)bh * DK + 2 * j) * dv + c0 + c] : 0.f;
        Sim[idx] = S0 ? S0[((size_t)bh * DK + 2 * j + 1) * dv + c0 + c] : 0.f;
    }

    const int n_chunks = (T_ + C - 1) / C;
    for (int ci = 0; ci < n_chunks; ++ci) {
        const int t0 = ci * C;
        const int len = min(C, T_ - t0);
        __syncthreads();
        load_and_rotate<DK, C, T>(sm, k, q, alpha, theta, beta, nullptr, b, h, T_, H, t0, len);
        // the two decay weights every product with the state needs, once per chunk instead of once per use
        for (int idx = tid; idx < C * M; idx += kThreads) {
            const int t = idx / M, j = idx % M;
            const float l = sm.lg[t * SM::LS + j];
            aw[t * SM::LS + j] = expf(l);
            yw[t * SM::LS + j] = expf(sm.lgC[j] - l);
        }
        __syncthreads();

        // Gram blocks Kt (i < t) and Aq (i <= t).
        for (int p = tid; p < C * (C + 1) / 2; p += kThreads) {
            int t, i;
            tri_decode(p, &t, &i);
            float kr_ = 0.f, ki_ = 0.f, ar_ = 0.f, ai_ = 0.f;
            const float *kt = sm.kp + t * SM::KS, *ki = sm.kp + i * SM::KS, *qt = sm.qp + t * SM::KS;
            const float *lt = sm.lg + t * SM::LS, *li = sm.lg + i * SM::LS;
            for (int j = 0; j < M; ++j) {
                const float w = expf(lt[j] - li[j]);
                const float br = w * ki[2 * j], bi = w * ki[2 * j + 1];
                const float xr = kt[2 * j], xi = kt[2 * j + 1];
                kr_ += xr * br + xi * bi;   // conj(x) * b
                ki_ += xr * bi - xi * br;
                const float yr = qt[2 * j], yi = qt[2 * j + 1];
                ar_ += yr * br + yi * bi;
                ai_ += yr * bi - yi * br;
            }
            Ktr[t * SM::GS + i] = kr_;
            Kti[t * SM::GS + i] = ki_;
            Aqr[t * SM::GS + i] = ar_;
            Aqi[t * SM::GS + i] = ai_;
        }

        // R = V - W^* S_0 (kept in E).
        for (int t = wid; t < C; t += kThreads / 32) {
            float rr = 0.f, ri = 0.f;
            if (t < len) rr = ld_val(v, (((size_t)b * T_ + t0 + t) * H + h) * dv + c0 + lane);
            const float *kt = sm.kp + t * SM::KS, *at = aw + t * SM::LS;
            for (int j = 0; j < M; ++j) {
                const float w = at[j];
                const float wr = w * kt[2 * j], wi = w * kt[2 * j + 1];
                const float sr = Sre[j * kSlice + lane], si = Sim[j * kSlice + lane];
                rr -= wr * sr + wi * si;   // conj(w) * s
                ri -= wr * si - wi * sr;
            }
            Er[t * kSlice + lane] = rr;
            Ei[t * kSlice + lane] = ri;
        }
        __syncthreads();

        // Forward substitution of (I + D_beta Kt) E = D_beta R.  A warp owns four columns; the sum
        // over earlier tokens is split over eight lanes and folded with shuffles.
        {
            const int cc = 4 * wid + lane / 8, part = lane % 8;
            for (int t = 0; t < C; ++t) {
                float sr = 0.f, si = 0.f;
                for (int i = part; i < t; i += 8) {
                    const float xr = Ktr[t * SM::GS + i], xi = Kti[t * SM::GS + i];
                    const float er = Er[i * kSlice + cc], ei = Ei[i * kSlice + cc];
                    sr += xr * er - xi * ei;
                    si += xr * ei + xi * er;
                }
#pragma unroll
                for (int off = 1; off < 8; off <<= 1) {
                    sr += __shfl_xor_sync(0xffffffffu, sr, off);
                    si += __shfl_xor_sync(0xffffffffu, si, off);
                }
                const float bt = sm.beta[t];
                const float er = bt * (Er[t * kSlice + cc] - sr);
                const float ei = bt * (Ei[t * kSlice + cc] - si);
                __syncwarp();
                if (part == 0) {
                    Er[t * kSlice + cc] = er;
                    Ei[t * kSlice + cc] = ei;
                }
                __syncwarp();
            }
        }
        __syncthreads();

        // Outputs: o_t^* = (conj(gamma_t) q_t)^* S_0 + sum_{i<=t} Aq[t][i] e_i^T ; o = conj of that row.
        for (int t = wid; t < len; t += kThreads / 32) {
            float rr = 0.f, ri = 0.f;
            const float *qt = sm.qp + t * SM::KS, *at = aw + t * SM::LS;
            for (int j = 0; j < M; ++j) {
                const float w = at[j];
                const float wr = w * qt[2 * j], wi = w * qt[2 * j + 1];
                const float sr = Sre[j * kSlice + lane], si = Sim[j * kSlice + lane];
                rr += wr * sr + wi * si;
                ri += wr * si - wi * sr;
            }
            for (int i = 0; i <= t; ++i) {
                const float xr = Aqr[t * SM::GS + i], xi = Aqi[t * SM::GS + i];
                const float er = Er[i * kSlice + lane], ei = Ei[i * kSlice + lane];
                rr += xr * er - xi * ei;
                ri += xr * ei + xi * er;
            }
            const size_t g = (((size_t)b * T_ + t0 + t) * H + h) * dv + c0 + lane;
            st_val(o, g, rr);
            if (o_im) st_val(o_im, g, -ri);
        }
        __syncthreads();

        // S_C = Gamma_C S_0 + sum_t (gamma_C / gamma_t) k_t e_t^T.
        for (int j = wid; j < M; j += kThreads / 32) {
            const float aC = expf(sm.lgC[j]);
            float nr = aC * Sre[j * kSlice + lane], ni = aC * Sim[j * kSlice + lane];
            for (int t = 0; t < C; ++t) {
                const float w = yw[t * SM::LS + j];
                const float yr = w * sm.kp[t * SM::KS + 2 * j], yi = w * sm.kp[t * SM::KS + 2 * j + 1];
                const float er = Er[t * kSlice + lane], ei = Ei[t * kSlice + lane];
                nr += yr * er - yi * ei;
                ni += yr * ei + yi * er;
            }
            const float gr = sm.gcr[j], gi = sm.gci[j];   // e^{i phi_C}
            Sre[j * kSlice + lane] = gr * nr - gi * ni;
            Sim[j * kSlice + lane] = gr * ni + gi * nr;
        }
    }
    __syncthreads();
    if (S_T) {
        for (int idx = tid; idx < M * kSlice; idx += kThreads) {
            const int j = idx / kSlice, c = idx % kSlice;
            S_T[((size_t)bh * DK + 2 * j) * dv + c0 + c] = Sre[idx];
            S_T[((size_t)bh * DK + 2 * j + 1) * dv + c0 + c] = Sim[idx];
        }
    }
}

// ------------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------------
template <int DK, int C, typename T>
cudaError_t launch_fwd(const ForwardArgs &a, cudaStream_t stream)
{
    constexpr size_t smem = sizeof(float) * forward_smem_floats<DK, C>();
    auto kern = sfda_forward_simt_kernel<DK, C, T>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)a.B * a.H * (a.d_v / kSlice);
    kern<<<grid, kThreads, smem, stream>>>(static_cast<const T *>(a.q), static_cast<const T *>(a.k),
                                           static_cast<const T *>(a.v), a.alpha, a.theta, a.beta, a.S0,
                                           static_cast<T *>(a.o), static_cast<T *>(a.o_im), a.S_T, a.T, a.H,
                                           a.d_v);
    return cudaGetLastError();
}

template <typename Args, typename T, typename F64_16, typename F64_32, typename F64_64, typename F128_16,
          typename F128_32, typename F128_64>
cudaError_t by_shape(const Args &a, F64_16 f1, F64_32 f2, F64_64 f3, F128_16 f4, F128_32 f5, F128_64 f6)
{
    if (a.d_k == 64 && a.chunk == 16) return f1();
    if (a.d_k == 64 && a.chunk == 32) return f2();
    if (a.d_k == 64 && a.chunk == 64) return f3();
    if (a.d_k == 128 && a.chunk == 16) return f4();
    if (a.d_k == 128 && a.chunk == 32) return f5();
    if (a.d_k == 128 && a.chunk == 64) return f6();
    return cudaErrorInvalidValue;
}

template <typename T>
cudaError_t dispatch_fwd(const ForwardArgs &a, cudaStream_t s)
{
    return by_shape<ForwardArgs, T>(
        a, [&] { return launch_fwd<64, 16, T>(a, s); }, [&] { return launch_fwd<64, 32, T>(a, s); },
        [&] { return launch_fwd<64, 64, T>(a, s); }, [&] { return launch_fwd<128, 16, T>(a, s); },
        [&] { return launch_fwd<128, 32, T>(a, s); }, [&] { return launch_fwd<128, 64, T>(a, s); });
}

}  // namespace

cudaError_t launch_forward_simt(const ForwardArgs &a, cudaStream_t stream, int *launches)
{
    const cudaError_t e = a.dtype == 1 ? dispatch_fwd<__nv_bfloat16>(a, stream) : dispatch_fwd<float>(a, stream);
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace sfda
