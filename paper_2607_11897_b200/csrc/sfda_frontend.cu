// sfda_frontend: the stable parameterisation of Section 3 as a kernel of its own,
//
//     alpha = alpha_min + (alpha_max - alpha_min) sigmoid(a)      (Eq. "param-alpha")
//     theta = theta_max tanh(b)                                   (Eq. "param-theta")
//     beta  = sigmoid(c)                                          (Eq. "param-beta")
//     k     = k_raw / (|k_raw|_2 + eps)                           (Eq. "param-key")
//
// for callers that want the four arrays themselves, and for the shapes whose forward runs on the CUDA cores.
// (The tensor-core forward applies the same map inside its operand preparation and never writes these arrays.)
//
// HBM-bound: every element is read once and written once.  One warp owns a (token, head) row -- d_k real key
// channels, d_k / 2 decay and phase coordinates, one beta -- so the key's norm is a shuffle reduction, every access
// is a coalesced vector load or store, and a warp keeps kRowsPerWarp rows in flight to cover the memory latency.
#include "sfda_common.cuh"
#include "sfda_internal.h"

namespace sfda {
namespace {

constexpr int kFrontThreads = 256;
constexpr int kRowsPerWarp = 4;

template <typename T, int N>
struct alignas(sizeof(T) * N) Vec {
    T x[N];
};

template <int DK, typename T>
__global__ void __launch_bounds__(kFrontThreads)
sfda_frontend_kernel(const float *__restrict__ a_raw, const float *__restrict__ b_raw, const float *__restrict__ c_raw,
                     const T *__restrict__ k_raw, float *__restrict__ alpha, float *__restrict__ theta,
                     float *__restrict__ beta, T *__restrict__ k, long long rows, float a_lo, float a_range,
                     float th_max, float eps)
{
    constexpr int CPL = DK / 32;      // real key channels per lane
    constexpr int MPL = CPL / 2;      // decay / phase coordinates per lane
    using KV = Vec<T, CPL>;
    using FV = Vec<float, MPL>;
    const int lane = threadIdx.x & 31;
    const long long warp = (long long)blockIdx.x * (kFrontThreads / 32) + (threadIdx.x >> 5);
    const long long n_warps = (long long)gridDim.x * (kFrontThreads / 32);

    for (long long r0 = warp * kRowsPerWarp; r0 < rows; r0 += n_warps * kRowsPerWarp) {
        KV kv[kRowsPerWarp];
        FV av[kRowsPerWarp], bv[kRowsPerWarp];
        float cv[kRowsPerWarp];
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) {
            const long long r = r0 + i;
            if (r < rows) {
                kv[i] = reinterpret_cast<const KV *>(k_raw + r * DK)[lane];
                av[i] = reinterpret_cast<const FV *>(a_raw + r * (DK / 2))[lane];
                bv[i] = reinterpret_cast<const FV *>(b_raw + r * (DK / 2))[lane];
                cv[i] = c_raw[r];
            }
        }
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) {
            const long long r = r0 + i;
            if (r >= rows) break;                    // uniform over the warp
            float kf[CPL], ss = 0.f;
#pragma unroll
            for (int x = 0; x < CPL; ++x) {
                kf[x] = ld_val(kv[i].x, x);
                ss = fmaf(kf[x], kf[x], ss);
            }
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
            // (a zero key with eps = 0 maps to a zero key)
            const float sk = 1.0f / fmaxf(sqrtf(ss) + eps, 1.0e-30f);
            KV ko;
            FV ao, to;
#pragma unroll
            for (int x = 0; x < CPL; ++x) st_val(ko.x, x, kf[x] * sk);
#pragma unroll
            for (int x = 0; x < MPL; ++x) {
                ao.x[x] = fmaf(a_range, 1.0f / (1.0f + expf(-av[i].x[x])), a_lo);
                to.x[x] = th_max * tanhf(bv[i].x[x]);
            }
            reinterpret_cast<KV *>(k + r * DK)[lane] = ko;
            reinterpret_cast<FV *>(alpha + r * (DK / 2))[lane] = ao;
            reinterpret_cast<FV *>(theta + r * (DK / 2))[lane] = to;
            if (lane == 0) beta[r] = 1.0f / (1.0f + expf(-cv[i]));
        }
    }
}

// The derivative of the same map: gradients with respect to alpha, theta, beta, k in, gradients with respect to the
// raw inputs out,
//
//     da = dalpha (alpha_max - alpha_min) sigmoid(a) (1 - sigmoid(a))      db = dtheta theta_max (1 - tanh(b)^2)
//     dc = dbeta sigmoid(c) (1 - sigmoid(c))       dk_raw = s dk - s^2 (dk . k_raw) k_raw / |k_raw|,  s = 1 / (|k_raw| + eps)
//
// (a zero key passes s dk through).  Same mapping of warps to rows; HBM-bound: two reads and one write of the
// forward's arrays.
template <int DK, typename T>
__global__ void __launch_bounds__(kFrontThreads)
sfda_frontend_backward_kernel(const float *__restrict__ a_raw, const float *__restrict__ b_raw,
                              const float *__restrict__ c_raw, const T *__restrict__ k_raw,
                              const float *__restrict__ dalpha, const float *__restrict__ dtheta,
                              const float *__restrict__ dbeta, const T *__restrict__ dk, float *__restrict__ da,
                              float *__restrict__ db, float *__restrict__ dc, T *__restrict__ dk_raw, long long rows,
                              float a_range, float th_max, float eps)
{
    constexpr int CPL = DK / 32, MPL = CPL / 2;
    using KV = Vec<T, CPL>;
    using FV = Vec<float, MPL>;
    constexpr int kRows = 2;          // rows in flight per warp (four were slower: 1.27 ms against 0.97 ms)
    const int lane = threadIdx.x & 31;
    const long long warp = (long long)blockIdx.x * (kFrontThreads / 32) + (threadIdx.x >> 5);
    const long long n_warps = (long long)gridDim.x * (kFrontThreads / 32);
    for (long long r0 = warp * kRows; r0 < rows; r0 += n_warps * kRows) {
        KV kv[kRows], gv[kRows];
        FV av[kRows], bv[kRows], gav[kRows], gbv[kRows];
        float cv[kRows], gcv[kRows];
#pragma unroll
        for (int i = 0; i < kRows; ++i) {
            const long long r = r0 + i;
            if (r < rows) {
                kv[i] = reinterpret_cast<const KV *>(k_raw + r * DK)[lane];
                gv[i] = reinterpret_cast<const KV *>(dk + r * DK)[lane];
                av[i] = reinterpret_cast<const FV *>(a_raw + r * (DK / 2))[lane];
                bv[i] = reinterpret_cast<const FV *>(b_raw + r * (DK / 2))[lane];
                gav[i] = reinterpret_cast<const FV *>(dalpha + r * (DK / 2))[lane];
                gbv[i] = reinterpret_cast<const FV *>(dtheta + r * (DK / 2))[lane];
                cv[i] = c_raw[r];
                gcv[i] = dbeta[r];
            }
        }
#pragma unroll
        for (int i = 0; i < kRows; ++i) {
            const long long r = r0 + i;
            if (r >= rows) break;                    // uniform over the warp
            float kf[CPL], gf[CPL], ss = 0.f, dot = 0.f;
#pragma unroll
            for (int x = 0; x < CPL; ++x) {
                kf[x] = ld_val(kv[i].x, x);
                gf[x] = ld_val(gv[i].x, x);
                ss = fmaf(kf[x], kf[x], ss);
                dot = fmaf(gf[x], kf[x], dot);
            }
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) {
                ss += __shfl_xor_sync(0xffffffffu, ss, d);
                dot += __shfl_xor_sync(0xffffffffu, dot, d);
            }
            const float n = sqrtf(ss);
            const float s = 1.0f / fmaxf(n + eps, 1.0e-30f);
            const float w = n > 0.f ? s * s * dot / n : 0.f;
            KV ko;
            FV ao, bo;
#pragma unroll
            for (int x = 0; x < CPL; ++x) st_val(ko.x, x, fmaf(s, gf[x], -w * kf[x]));
#pragma unroll
            for (int x = 0; x < MPL; ++x) {
                const float sg = 1.0f / (1.0f + expf(-av[i].x[x]));
                const float th = tanhf(bv[i].x[x]);
                ao.x[x] = gav[i].x[x] * a_range * sg * (1.0f - sg);
                bo.x[x] = gbv[i].x[x] * th_max * (1.0f - th * th);
            }
            reinterpret_cast<KV *>(dk_raw + r * DK)[lane] = ko;
            reinterpret_cast<FV *>(da + r * (DK / 2))[lane] = ao;
            reinterpret_cast<FV *>(db + r * (DK / 2))[lane] = bo;
            if (lane == 0) {
                const float sg = 1.0f / (1.0f + expf(-cv[i]));
                dc[r] = gcv[i] * sg * (1.0f - sg);
            }
        }
    }
}

template <int DK, typename T>
cudaError_t launch_typed(const FrontendArgs &a, cudaStream_t stream, int *launches)
{
    const long long rows_per_block = (long long)(kFrontThreads / 32) * kRowsPerWarp;
    long long blocks = (a.rows + rows_per_block - 1) / rows_per_block;
    int dev = 0, n_sm = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const long long cap = (long long)n_sm * 8 * 4;      // a few waves of resident blocks, then the grid strides
    if (blocks > cap) blocks = cap;
    if (a.backward)
        sfda_frontend_backward_kernel<DK, T><<<(unsigned)blocks, kFrontThreads, 0, stream>>>(
            a.a_raw, a.b_raw, a.c_raw, static_cast<const T *>(a.k_raw), a.dalpha, a.dtheta, a.dbeta,
            static_cast<const T *>(a.dk), a.alpha, a.theta, a.beta, static_cast<T *>(a.k), a.rows,
            a.alpha_max - a.alpha_min, a.theta_max, a.eps);
    else
        sfda_frontend_kernel<DK, T><<<(unsigned)blocks, kFrontThreads, 0, stream>>>(
            a.a_raw, a.b_raw, a.c_raw, static_cast<const T *>(a.k_raw), a.alpha, a.theta, a.beta, static_cast<T *>(a.k),
            a.rows, a.alpha_min, a.alpha_max - a.alpha_min, a.theta_max, a.eps);
    e = cudaGetLastError();
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace

cudaError_t launch_frontend(const FrontendArgs &a, cudaStream_t stream, int *launches)
{
    if (a.dtype == 1)
        return a.d_k == 128 ? launch_typed<128, __nv_bfloat16>(a, stream, launches)
                            : launch_typed<64, __nv_bfloat16>(a, stream, launches);
    return a.d_k == 128 ? launch_typed<128, float>(a, stream, launches) : launch_typed<64, float>(a, stream, launches);
}

}  // namespace sfda
