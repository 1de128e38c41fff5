// sfda_backward: reverse-mode derivative of the recurrence of Section 3 (Eq. "sfda") with o_t = S_t^* q_t, token by
// token in fp32 on the CUDA cores.  (The paper asks for the backward pass only as something to be timed, App. E; what
// it computes is the adjoint of Eq. "sfda".)  This is the first correct path: one CTA per (batch, head) pair and
// block of value columns (the columns of the state and of its cotangent never interact; with many sequences a block
// is all d_v columns, with few it is 64 or 32 of them so that every SM has work) walks the sequence three times --
//
//   1. forward, keeping the state at the start of every segment of kSeg tokens (checkpoints in the workspace);
//   2. per segment, last to first: forward again from the checkpoint, keeping S_{t-1} of every token of the segment;
//   3. backward through the segment with the cotangent G of the state in shared memory.
//
// One backward step, with Z = Lambda_t S_{t-1}, u^T = v_t^T - k_t^* Z (so S_t = Z + beta_t k_t u^T) and
// yb_t = do_re + i do_im:
//
//   G += q yb^*                    p = G^* k                     dv = beta Re p            dbeta = Re(u^T p)
//   dq = Z yb + beta k (u^T yb)    dk = beta (G conj(u) - Z p)   Zb = G - beta k p^*
//   lamb_j = sum_c conj(S_{t-1,jc}) Zb_jc      dalpha = Re(conj(lamb) e^{i theta})     dtheta = -Im(conj(lamb) lam)
//   G <- conj(lam) Zb   (row-wise: the cotangent of S_{t-1})
//
// Complex cotangents Xb mean dL = Re sum conj(Xb) dX, i.e. the ordinary gradient with respect to the (Re, Im) pair.
// dq, dk, dalpha, dtheta, dbeta are sums over the value columns: with more than one column block every block writes
// its share as fp32 to the workspace and a second kernel adds the shares in a fixed order, so the result is
// deterministic either way.
#include "sfda_common.cuh"
#include "sfda_internal.h"

namespace sfda {
namespace {

constexpr int kBwdThreads = 512;
constexpr int kSeg = 64;     // tokens between checkpoints

template <int DK, int DV>
struct BwdSmem {
    static constexpr int M = DK / 2;
    static constexpr int RS = DV + 8;            // row stride in complex (float2) elements: rows 16 banks apart
    static constexpr int NG = kBwdThreads / DV;  // row groups of the column-owner mapping
    static constexpr int plane = M * RS;         // floats in half a state buffer
    // G and two buffers of S_{t-1} as interleaved complex [M][RS], and the vectors of one token
    static constexpr size_t bytes = (size_t)(6 * plane + 8 * M + 7 * DV + NG * 4 * DV + 64) * 4;
};

__device__ __forceinline__ void cp_async16(float *dst_smem, const float *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

struct BwdArgsDev {
    const void *q, *k, *v, *d_o, *d_o_im;
    const float *alpha, *theta, *beta, *S0, *dS_T;
    void *dq, *dk, *dv;
    float *dalpha, *dtheta, *dbeta, *dS0;
    float *dq_p, *dk_p, *dalpha_p, *dtheta_p, *dbeta_p;   // shares of the column blocks: [blocks][rows][...] fp32
    float *check, *scratch;      // [BH][blocks][NS][M][cols][2], [BH][blocks][kSeg][M][cols][2] (interleaved complex)
    size_t rows;                 // B * T * H
    int T, H, NS;
};

// DVT value columns per state, DV of them per CTA
template <int DK, int DVT, int DV, typename T>
__global__ void __launch_bounds__(kBwdThreads, 1)
sfda_backward_kernel(const BwdArgsDev a)
{
    constexpr int NSL = DVT / DV;                  // column blocks per state
    static_assert(DVT % DV == 0 && DV % 32 == 0, "the value columns split into blocks of whole warps");
    using L = BwdSmem<DK, DV>;
    constexpr int M = L::M, RS = L::RS, NG = L::NG, RA = M / NG;      // RA rows per thread in the column mapping
    constexpr int TPR = kBwdThreads / M, CPT = DV / TPR;               // threads per row / columns per thread (row mapping)
    static_assert(M % NG == 0 && DV % TPR == 0 && M + DV + 1 <= kBwdThreads, "thread mappings");
    extern __shared__ __align__(16) float sm[];
    float2 *G = reinterpret_cast<float2 *>(sm);            // cotangent of the state, complex [M][RS]
    float *P0 = sm + 2 * L::plane;                          // two buffers of the same shape for S / S_{t-1}
    auto Pb = [&](int i) { return reinterpret_cast<float2 *>(P0 + i * 2 * L::plane); };
    // per-row vectors of the token, packed so that one (broadcast) load fetches all a step needs of a row:
    // (lam re, lam im, k re, k im), (q re, q im, cos theta, sin theta); per-column vectors likewise:
    // (yb re, yb im, u re, u im), (p re, p im), v
    float4 *v_lk = reinterpret_cast<float4 *>(P0 + 4 * L::plane);
    float4 *v_qc = v_lk + M;
    float4 *v_yu = v_qc + M;
    float2 *v_p = reinterpret_cast<float2 *>(v_yu + DV);
    float *v_v = reinterpret_cast<float *>(v_p + DV);
    float *red = v_v + DV;                      // [NG][4][DV]
    float *scal = red + NG * 4 * DV;            // [0] beta, [8 + 4 w + x] partial sums of warp w

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bh = blockIdx.x, h = bh % a.H, b = bh / a.H, slice = blockIdx.y, c0 = slice * DV;
    const int T_ = a.T, H = a.H;
    const T *q = static_cast<const T *>(a.q), *k = static_cast<const T *>(a.k), *v = static_cast<const T *>(a.v);
    const T *d_o = static_cast<const T *>(a.d_o), *d_oi = static_cast<const T *>(a.d_o_im);
    float *check = a.check + ((size_t)bh * NSL + slice) * a.NS * 2 * M * DV;
    float *scratch = a.scratch + ((size_t)bh * NSL + slice) * kSeg * 2 * M * DV;

    // column-owner mapping (A): column c, rows g, g + NG, ...;  row-owner mapping (B): row jb, columns part + TPR n
    const int c = tid % DV, g = tid / DV;
    const int jb = tid / TPR, part = tid % TPR;

    // ---- token vectors: registers -> shared memory, one token ahead of the step that uses them
    float r0 = 0.f, r1 = 0.f, r2 = 0.f, r3 = 0.f, r4 = 0.f, r5 = 0.f;
    auto load_tok = [&](int t, bool back) {
        if (t < 0 || t >= T_) return;
        const size_t row = ((size_t)b * T_ + t) * H + h;
        if (tid < M) {
            r0 = a.alpha[row * M + tid];
            r1 = a.theta[row * M + tid];
            r2 = ld_val(k, row * DK + 2 * tid);
            r3 = ld_val(k, row * DK + 2 * tid + 1);
            if (back) {
                r4 = ld_val(q, row * DK + 2 * tid);
                r5 = ld_val(q, row * DK + 2 * tid + 1);
            }
        } else if (tid < M + DV) {
            const int cc = tid - M;
            r0 = ld_val(v, row * DVT + c0 + cc);
            if (back) {
                r1 = ld_val(d_o, row * DVT + c0 + cc);
                r2 = d_oi ? ld_val(d_oi, row * DVT + c0 + cc) : 0.f;
            }
        } else if (tid == M + DV) {
            r0 = a.beta[row];
        }
    };
    auto stage_tok = [&](bool back) {
        if (tid < M) {
            float sn, cs;
            sincosf(r1, &sn, &cs);
            v_lk[tid] = make_float4(r0 * cs, r0 * sn, r2, r3);
            if (back) v_qc[tid] = make_float4(r4, r5, cs, sn);
        } else if (tid < M + DV) {
            const int cc = tid - M;
            v_v[cc] = r0;
            if (back) v_yu[cc] = make_float4(r1, r2, 0.f, 0.f);
        } else if (tid == M + DV) {
            scal[0] = r0;
        }
    };

    // ---- one forward step on the state S; the token's vectors are staged and synchronised
    auto fwd_step = [&](float2 *S) {
        float cr = 0.f, ci = 0.f, zr[RA], zi[RA];
#pragma unroll
        for (int r = 0; r < RA; ++r) {
            const int j = g + NG * r;
            const float4 lk = v_lk[j];
            const float2 sv = S[j * RS + c];
            zr[r] = lk.x * sv.x - lk.y * sv.y;                                 // Z = Lambda S
            zi[r] = lk.x * sv.y + lk.y * sv.x;
            cr += lk.z * zr[r] + lk.w * zi[r];                                 // conj(k) z
            ci += lk.z * zi[r] - lk.w * zr[r];
        }
        red[(g * 4 + 0) * DV + c] = cr;
        red[(g * 4 + 1) * DV + c] = ci;
        __syncthreads();
        float sr_ = 0.f, si_ = 0.f;
#pragma unroll
        for (int gg = 0; gg < NG; ++gg) {
            sr_ += red[(gg * 4 + 0) * DV + c];
            si_ += red[(gg * 4 + 1) * DV + c];
        }
        const float bt = scal[0];
        const float er = bt * (v_v[c] - sr_), ei = -bt * si_;                  // e = beta u, u = v - k^* Z
#pragma unroll
        for (int r = 0; r < RA; ++r) {
            const int j = g + NG * r;
            const float4 lk = v_lk[j];
            S[j * RS + c] = make_float2(zr[r] + lk.z * er - lk.w * ei, zi[r] + lk.z * ei + lk.w * er);
        }
        __syncthreads();
    };

    // ---- state moves between shared and global memory (workspace format: interleaved complex [M][DV]), 16 bytes
    // = two elements per access
    auto store_state = [&](const float2 *S, float *dst) {
        for (int idx = tid; idx < M * DV / 2; idx += kBwdThreads) {
            const int j = idx / (DV / 2), c2 = idx % (DV / 2);
            *reinterpret_cast<float4 *>(dst + ((size_t)j * DV + 2 * c2) * 2) = *reinterpret_cast<const float4 *>(S + j * RS + 2 * c2);
        }
    };
    auto load_state_async = [&](float2 *S, const float *src) {
        for (int idx = tid; idx < M * DV / 2; idx += kBwdThreads) {
            const int j = idx / (DV / 2), c2 = idx % (DV / 2);
            cp_async16(reinterpret_cast<float *>(S + j * RS + 2 * c2), src + ((size_t)j * DV + 2 * c2) * 2);
        }
        cp_async_commit();
    };

    // ---- sweep 1: forward, checkpoints at the start of every segment (nothing is needed beyond the last one)
    float2 *S = Pb(0);
    for (int idx = tid; idx < M * DV; idx += kBwdThreads) {
        const int j = idx / DV, cc = idx % DV;
        S[j * RS + cc] = a.S0 ? make_float2(a.S0[((size_t)bh * DK + 2 * j) * DVT + c0 + cc], a.S0[((size_t)bh * DK + 2 * j + 1) * DVT + c0 + cc])
                              : make_float2(0.f, 0.f);
    }
    const int t_last_check = (a.NS - 1) * kSeg;
    load_tok(0, false);
    __syncthreads();
    for (int t = 0; t < t_last_check; ++t) {
        if (t % kSeg == 0) store_state(S, check + (size_t)(t / kSeg) * 2 * M * DV);
        stage_tok(false);
        __syncthreads();
        load_tok(t + 1, false);
        fwd_step(S);
    }
    store_state(S, check + (size_t)(a.NS - 1) * 2 * M * DV);

    // ---- cotangent of the final state
    for (int idx = tid; idx < M * DV; idx += kBwdThreads) {
        const int j = idx / DV, cc = idx % DV;
        G[j * RS + cc] = a.dS_T ? make_float2(a.dS_T[((size_t)bh * DK + 2 * j) * DVT + c0 + cc], a.dS_T[((size_t)bh * DK + 2 * j + 1) * DVT + c0 + cc])
                                : make_float2(0.f, 0.f);
    }
    __syncthreads();      // also: every thread's checkpoint stores precede the loads below (same CTA, after a barrier)

    T *dq = static_cast<T *>(a.dq), *dk = static_cast<T *>(a.dk), *dv = static_cast<T *>(a.dv);
    float *dq_p = a.dq_p + (size_t)slice * a.rows * DK, *dk_p = a.dk_p + (size_t)slice * a.rows * DK;
    float *dal_p = a.dalpha_p + (size_t)slice * a.rows * M, *dth_p = a.dtheta_p + (size_t)slice * a.rows * M;
    float *dbe_p = a.dbeta_p + (size_t)slice * a.rows;
    for (int si = a.NS - 1; si >= 0; --si) {
        const int t0 = si * kSeg, t1 = min(t0 + kSeg, T_);
        // ---- sweep 2: forward again from the checkpoint, S_{t-1} of every token to the scratch
        load_state_async(S, check + (size_t)si * 2 * M * DV);
        load_tok(t0, false);
        cp_async_wait_all();
        __syncthreads();
        for (int t = t0; t < t1; ++t) {
            store_state(S, scratch + (size_t)(t - t0) * 2 * M * DV);
            stage_tok(false);
            __syncthreads();
            load_tok(t + 1 < t1 ? t + 1 : t1 - 1, t + 1 >= t1);     // after the last one: the first backward token
            if (t + 1 < t1) fwd_step(S);                        // the state after the last token is not needed
        }
        __syncthreads();      // the scratch stores of this CTA are visible to its own later loads

        // ---- sweep 3: backward through the segment; S_{t-1} arrives one token ahead in the other buffer
        int buf = 0;
        load_state_async(Pb(buf), scratch + (size_t)(t1 - 1 - t0) * 2 * M * DV);
        for (int t = t1 - 1; t >= t0; --t) {
            stage_tok(true);
            cp_async_wait_all();
            __syncthreads();
            const float2 *Q = Pb(buf);
            if (t > t0) load_state_async(Pb(buf ^ 1), scratch + (size_t)(t - 1 - t0) * 2 * M * DV);
            load_tok(t - 1 >= t0 ? t - 1 : t0 - 1, true);           // (a token of the next segment down is reloaded there)
            const float bt = scal[0];
            const size_t row = ((size_t)b * T_ + t) * H + h;

            // step 1 (columns): partial p = (G + q yb^*)^* k and k^* Z  (G itself is updated in step 3)
            {
                const float4 yu = v_yu[c];
                const float yr = yu.x, yi = yu.y;
                float pr = 0.f, pi = 0.f, zr_ = 0.f, zi_ = 0.f;
#pragma unroll
                for (int r = 0; r < RA; ++r) {
                    const int j = g + NG * r;
                    const float4 lk = v_lk[j], qc = v_qc[j];
                    const float2 gv = G[j * RS + c];
                    const float gr = gv.x + qc.x * yr + qc.y * yi;              // G + q conj(yb)
                    const float gi = gv.y + qc.y * yr - qc.x * yi;
                    pr += gr * lk.z + gi * lk.w;                                // conj(G) k
                    pi += gr * lk.w - gi * lk.z;
                    const float2 sv = Q[j * RS + c];
                    const float zr = lk.x * sv.x - lk.y * sv.y, zi = lk.x * sv.y + lk.y * sv.x;
                    zr_ += lk.z * zr + lk.w * zi;                               // conj(k) z
                    zi_ += lk.z * zi - lk.w * zr;
                }
                red[(g * 4 + 0) * DV + c] = pr;
                red[(g * 4 + 1) * DV + c] = pi;
                red[(g * 4 + 2) * DV + c] = zr_;
                red[(g * 4 + 3) * DV + c] = zi_;
            }
            __syncthreads();
            // step 2: p, u per column; dv; the sums over columns u^T p and u^T yb
            if (tid < DV) {
                float pr = 0.f, pi = 0.f, zr = 0.f, zi = 0.f;
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) {
                    pr += red[(gg * 4 + 0) * DV + c];
                    pi += red[(gg * 4 + 1) * DV + c];
                    zr += red[(gg * 4 + 2) * DV + c];
                    zi += red[(gg * 4 + 3) * DV + c];
                }
                const float ur = v_v[c] - zr, ui = -zi;
                const float4 yu = v_yu[c];
                const float yr = yu.x, yi = yu.y;
                v_p[c] = make_float2(pr, pi);
                v_yu[c] = make_float4(yr, yi, ur, ui);
                st_val(dv, row * DVT + c0 + c, bt * pr);
                float s0 = ur * pr - ui * pi;                       // Re(u p)
                float s1 = ur * yr - ui * yi, s2 = ur * yi + ui * yr;   // u yb
#pragma unroll
                for (int d = 16; d >= 1; d >>= 1) {
                    s0 += __shfl_xor_sync(0xffffffffu, s0, d);
                    s1 += __shfl_xor_sync(0xffffffffu, s1, d);
                    s2 += __shfl_xor_sync(0xffffffffu, s2, d);
                }
                if (lane == 0) { scal[8 + 4 * warp] = s0; scal[9 + 4 * warp] = s1; scal[10 + 4 * warp] = s2; }
            }
            __syncthreads();
            // step 3 (rows): dq, dk, lamb, and G <- conj(lam) (G - beta k p^*)
            {
                float sr_ = 0.f, si_ = 0.f, dbe = 0.f;
#pragma unroll
                for (int w = 0; w < DV / 32; ++w) { dbe += scal[8 + 4 * w]; sr_ += scal[9 + 4 * w]; si_ += scal[10 + 4 * w]; }
                if (tid == 0) (NSL == 1 ? a.dbeta : dbe_p)[row] = dbe;
                const int j = jb;
                const float4 lk = v_lk[j], qc = v_qc[j];
                const float lr = lk.x, li = lk.y, kr = lk.z, ki = lk.w;
                float qzr = 0.f, qzi = 0.f, k1r = 0.f, k1i = 0.f, k2r = 0.f, k2i = 0.f, lbr = 0.f, lbi = 0.f;
#pragma unroll 4
                for (int n = 0; n < CPT; ++n) {
                    const int cc = part + TPR * n;
                    const float4 yu = v_yu[cc];
                    const float2 pp = v_p[cc];
                    const float yr = yu.x, yi = yu.y, ur = yu.z, ui = yu.w, pr = pp.x, pi = pp.y;
                    const float2 gv = G[j * RS + cc], sv = Q[j * RS + cc];
                    const float gr = gv.x + qc.x * yr + qc.y * yi;             // G + q conj(yb)
                    const float gi = gv.y + qc.y * yr - qc.x * yi;
                    const float sr = sv.x, si2 = sv.y;
                    const float zr = lr * sr - li * si2, zi = lr * si2 + li * sr;
                    qzr += zr * yr - zi * yi;  qzi += zr * yi + zi * yr;       // Z yb
                    k1r += gr * ur + gi * ui;  k1i += gi * ur - gr * ui;       // G conj(u)
                    k2r += zr * pr - zi * pi;  k2i += zr * pi + zi * pr;       // Z p
                    // Zb = G - beta k conj(p)
                    const float br = gr - bt * (kr * pr + ki * pi), bi = gi - bt * (ki * pr - kr * pi);
                    lbr += sr * br + si2 * bi;  lbi += sr * bi - si2 * br;     // conj(S_{t-1}) Zb
                    G[j * RS + cc] = make_float2(lr * br + li * bi, lr * bi - li * br);   // conj(lam) Zb
                }
#pragma unroll
                for (int d = TPR / 2; d >= 1; d >>= 1) {
                    qzr += __shfl_xor_sync(0xffffffffu, qzr, d);  qzi += __shfl_xor_sync(0xffffffffu, qzi, d);
                    k1r += __shfl_xor_sync(0xffffffffu, k1r, d);  k1i += __shfl_xor_sync(0xffffffffu, k1i, d);
                    k2r += __shfl_xor_sync(0xffffffffu, k2r, d);  k2i += __shfl_xor_sync(0xffffffffu, k2i, d);
                    lbr += __shfl_xor_sync(0xffffffffu, lbr, d);  lbi += __shfl_xor_sync(0xffffffffu, lbi, d);
                }
                if (part == 0) {
                    const float dqr = qzr + bt * (kr * sr_ - ki * si_), dqi = qzi + bt * (kr * si_ + ki * sr_);   // + beta k (u^T yb)
                    const float dkr = bt * (k1r - k2r), dki = bt * (k1i - k2i);
                    const float cs = qc.z, sn = qc.w;
                    const float dal = lbr * cs + lbi * sn;                                // Re(conj(lamb) e^{i theta})
                    const float dth = lbi * lr - lbr * li;                                // -Im(conj(lamb) lam)
                    if constexpr (NSL == 1) {
                        st_val(dq, row * DK + 2 * j, dqr);
                        st_val(dq, row * DK + 2 * j + 1, dqi);
                        st_val(dk, row * DK + 2 * j, dkr);
                        st_val(dk, row * DK + 2 * j + 1, dki);
                        a.dalpha[row * M + j] = dal;
                        a.dtheta[row * M + j] = dth;
                    } else {      // this column block's share of the sums over the columns
                        *reinterpret_cast<float2 *>(dq_p + row * DK + 2 * j) = make_float2(dqr, dqi);
                        *reinterpret_cast<float2 *>(dk_p + row * DK + 2 * j) = make_float2(dkr, dki);
                        dal_p[row * M + j] = dal;
                        dth_p[row * M + j] = dth;
                    }
                }
            }
            __syncthreads();
            buf ^= 1;
        }
        S = Pb(0);
    }
    for (int idx = tid; idx < M * DV; idx += kBwdThreads) {
        const int j = idx / DV, cc = idx % DV;
        a.dS0[((size_t)bh * DK + 2 * j) * DVT + c0 + cc] = G[j * RS + cc].x;
        a.dS0[((size_t)bh * DK + 2 * j + 1) * DVT + c0 + cc] = G[j * RS + cc].y;
    }
}

// ---- the sums over the column blocks: out[i] = share_0[i] + share_1[i] + ... in that order, one thread per four
// consecutive elements.  HBM-bound and small beside the sweeps.
constexpr int kSumThreads = 256;

__device__ __forceinline__ void st_val4(float *p, float4 x) { *reinterpret_cast<float4 *>(p) = x; }
__device__ __forceinline__ void st_val4(__nv_bfloat16 *p, float4 x)
{
    const __nv_bfloat162 lo = __floats2bfloat162_rn(x.x, x.y), hi = __floats2bfloat162_rn(x.z, x.w);
    *reinterpret_cast<uint2 *>(p) = make_uint2(*reinterpret_cast<const uint32_t *>(&lo), *reinterpret_cast<const uint32_t *>(&hi));
}

template <int NSL, typename T>
__global__ void __launch_bounds__(kSumThreads)
sfda_backward_sum_kernel(const float *__restrict__ dq_p, const float *__restrict__ dk_p, const float *__restrict__ dal_p,
                         const float *__restrict__ dth_p, const float *__restrict__ dbe_p, T *__restrict__ dq,
                         T *__restrict__ dk, float *__restrict__ dalpha, float *__restrict__ dtheta,
                         float *__restrict__ dbeta, size_t n_key, size_t n_coord, size_t rows)
{
    // work items in float4 units: [dq | dk | dalpha | dtheta] then dbeta one by one
    const size_t q4 = n_key / 4, c4 = n_coord / 4, total = 2 * q4 + 2 * c4 + rows;
    for (size_t i = (size_t)blockIdx.x * kSumThreads + threadIdx.x; i < total; i += (size_t)gridDim.x * kSumThreads) {
        if (i < 2 * q4 + 2 * c4) {
            const float *src;
            size_t n, at;
            int which;
            if (i < q4) { src = dq_p; n = n_key; at = i; which = 0; }
            else if (i < 2 * q4) { src = dk_p; n = n_key; at = i - q4; which = 1; }
            else if (i < 2 * q4 + c4) { src = dal_p; n = n_coord; at = i - 2 * q4; which = 2; }
            else { src = dth_p; n = n_coord; at = i - 2 * q4 - c4; which = 3; }
            float4 acc = *reinterpret_cast<const float4 *>(src + 4 * at);
#pragma unroll
            for (int sl = 1; sl < NSL; ++sl) {
                const float4 x = *reinterpret_cast<const float4 *>(src + (size_t)sl * n + 4 * at);
                acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
            }
            if (which >= 2) {
                *reinterpret_cast<float4 *>((which == 2 ? dalpha : dtheta) + 4 * at) = acc;
            } else {
                st_val4((which == 0 ? dq : dk) + 4 * at, acc);
            }
        } else {
            const size_t at = i - 2 * q4 - 2 * c4;
            float acc = dbe_p[at];
#pragma unroll
            for (int sl = 1; sl < NSL; ++sl) acc += dbe_p[(size_t)sl * rows + at];
            dbeta[at] = acc;
        }
    }
}

// Value columns per CTA: all of them while the (batch, head) pairs alone fill the SMs; halved (down to 32) while the
// grid still fits the SMs of a B200, so that few sequences use the whole device.  (A fixed count rather than the
// device's: the workspace size must not depend on where it is asked for.)
constexpr int kBwdTargetCtas = 148;

int bwd_cols(int B, int H, int d_v)
{
    int cols = d_v;
    while (cols > 32 && (long long)B * H * (d_v / (cols / 2)) <= kBwdTargetCtas) cols /= 2;
    return cols;
}

// workspace: checkpoints, the S_{t-1} of one segment, then (more than one column block only) the blocks' shares of
// dq, dk, dalpha, dtheta, dbeta
struct BwdWorkspace {
    size_t check, scratch, dq, dk, dalpha, dtheta, dbeta, total;   // offsets and size in floats
};

BwdWorkspace bwd_workspace(int B, int T, int H, int d_k, int d_v)
{
    const size_t bhn = (size_t)B * H, ns = (size_t)(T + kSeg - 1) / kSeg, state = (size_t)d_k * d_v;
    const size_t rows = bhn * T, nsl = (size_t)(d_v / bwd_cols(B, H, d_v)), shares = nsl > 1 ? nsl * rows : 0;
    BwdWorkspace w;
    w.check = 0;
    w.scratch = w.check + bhn * ns * state;
    w.dq = w.scratch + bhn * kSeg * state;
    w.dk = w.dq + shares * d_k;
    w.dalpha = w.dk + shares * d_k;
    w.dtheta = w.dalpha + shares * (d_k / 2);
    w.dbeta = w.dtheta + shares * (d_k / 2);
    w.total = w.dbeta + ((shares + 3) & ~(size_t)3);
    return w;
}

template <int DK, int DVT, int DV, typename T>
cudaError_t launch_cols(const BackwardArgs &x, void *workspace, cudaStream_t stream, int *launches)
{
    using L = BwdSmem<DK, DV>;
    constexpr int NSL = DVT / DV;
    auto kern = sfda_backward_kernel<DK, DVT, DV, T>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::bytes);
    if (e != cudaSuccess) return e;
    const BwdWorkspace w = bwd_workspace(x.B, x.T, x.H, DK, DVT);
    float *ws = static_cast<float *>(workspace);
    BwdArgsDev a;
    a.q = x.q; a.k = x.k; a.v = x.v; a.d_o = x.d_o; a.d_o_im = x.d_o_im;
    a.alpha = x.alpha; a.theta = x.theta; a.beta = x.beta; a.S0 = x.S0; a.dS_T = x.dS_T;
    a.dq = x.dq; a.dk = x.dk; a.dv = x.dv; a.dalpha = x.dalpha; a.dtheta = x.dtheta; a.dbeta = x.dbeta; a.dS0 = x.dS0;
    a.T = x.T; a.H = x.H; a.NS = (x.T + kSeg - 1) / kSeg;
    const size_t bhn = (size_t)x.B * x.H;
    a.rows = bhn * x.T;
    a.check = ws + w.check; a.scratch = ws + w.scratch;
    a.dq_p = ws + w.dq; a.dk_p = ws + w.dk; a.dalpha_p = ws + w.dalpha; a.dtheta_p = ws + w.dtheta; a.dbeta_p = ws + w.dbeta;
    kern<<<dim3((unsigned)bhn, NSL), kBwdThreads, L::bytes, stream>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (launches) ++*launches;
    if constexpr (NSL > 1) {
        const size_t n_key = a.rows * DK, n_coord = a.rows * (DK / 2);
        const size_t items = n_key / 2 + n_coord / 2 + a.rows;
        size_t blocks = (items + kSumThreads - 1) / kSumThreads;
        if (blocks > 148 * 8 * 8) blocks = 148 * 8 * 8;
        sfda_backward_sum_kernel<NSL, T><<<(unsigned)blocks, kSumThreads, 0, stream>>>(
            a.dq_p, a.dk_p, a.dalpha_p, a.dtheta_p, a.dbeta_p, static_cast<T *>(x.dq), static_cast<T *>(x.dk), x.dalpha,
            x.dtheta, x.dbeta, n_key, n_coord, a.rows);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        if (launches) ++*launches;
    }
    return cudaSuccess;
}

template <int DK, int DV, typename T>
cudaError_t launch_typed(const BackwardArgs &x, void *workspace, cudaStream_t stream, int *launches)
{
    const int cols = bwd_cols(x.B, x.H, DV);
    if (cols == DV) return launch_cols<DK, DV, DV, T>(x, workspace, stream, launches);
    if constexpr (DV > 64) {
        if (cols == 64) return launch_cols<DK, DV, 64, T>(x, workspace, stream, launches);
    }
    return launch_cols<DK, DV, 32, T>(x, workspace, stream, launches);
}

}  // namespace

size_t backward_workspace_bytes(int B, int T, int H, int d_k, int d_v)
{
    return bwd_workspace(B, T, H, d_k, d_v).total * sizeof(float);
}

cudaError_t launch_backward(const BackwardArgs &a, void *workspace, cudaStream_t stream, int *launches)
{
    cudaError_t e = cudaErrorInvalidValue;
    if (a.dtype == 1) {
        if (a.d_k == 128 && a.d_v == 128) e = launch_typed<128, 128, __nv_bfloat16>(a, workspace, stream, launches);
        else if (a.d_k == 128 && a.d_v == 64) e = launch_typed<128, 64, __nv_bfloat16>(a, workspace, stream, launches);
        else if (a.d_k == 64 && a.d_v == 128) e = launch_typed<64, 128, __nv_bfloat16>(a, workspace, stream, launches);
        else if (a.d_k == 64 && a.d_v == 64) e = launch_typed<64, 64, __nv_bfloat16>(a, workspace, stream, launches);
    } else {
        if (a.d_k == 128 && a.d_v == 128) e = launch_typed<128, 128, float>(a, workspace, stream, launches);
        else if (a.d_k == 128 && a.d_v == 64) e = launch_typed<128, 64, float>(a, workspace, stream, launches);
        else if (a.d_k == 64 && a.d_v == 128) e = launch_typed<64, 128, float>(a, workspace, stream, launches);
        else if (a.d_k == 64 && a.d_v == 64) e = launch_typed<64, 64, float>(a, workspace, stream, launches);
    }
    return e;
}

}  // namespace sfda
