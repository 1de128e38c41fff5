// sfda_backward: reverse-mode derivative of the recurrence of Section 3 (Eq. "sfda") with o_t = S_t^* q_t, token by
// token in fp32 on the CUDA cores.  (The paper asks for the backward pass only as something to be timed, App. E; what
// it computes is the adjoint of Eq. "sfda".)  This is the first correct path: one CTA per (batch, head) pair and
// block of value columns (the columns of the state and of its cotangent never interact; with many sequences a block
// is all d_v columns, with few it is 64 or 32 of them so that every SM has work) walks the sequence three times --
//
//   1. forward, keeping the state at the start of every segment of kSeg tokens (checkpoints in the workspace);
//   2. per segment, last to first: forward again from the checkpoint, keeping S_{t-1} of every token of the segment;
//   3. backward through the segment.
//
// The state (sweeps 1, 2) and its cotangent G (sweep 3) live in registers, a tile of rows x columns per thread;
// S_{t-1} of the backward step arrives from the scratch by cp.async, one token ahead.
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

// Thread mapping: warp w owns TR consecutive rows of the (complex) state, lane l owns TC consecutive value columns,
// so a thread keeps a TR x TC tile of the cotangent G -- and of the state, while a step needs it -- in registers.
// Sums over rows (per column) cross the warps through shared memory; sums over columns (per row) stay inside a warp.
template <int DK, int DV>
struct BwdSmem {
    static constexpr int M = DK / 2, NW = kBwdThreads / 32;
    static constexpr int TR = M / NW, TC = DV / 32;
    static_assert(M % NW == 0 && DV % 32 == 0 && (TC == 1 || TC == 2 || TC == 4), "tile shape");
    // two buffers of S_{t-1} (interleaved complex [M][DV]), the warps' partial column sums [NW][DV] float4, two
    // sets of token vectors (row vectors 2 float4 [M], column vectors float2 + float [DV], beta), and the
    // per-column results of a step (p, u / e: 2 float2 [DV]) with the warps' scalar sums
    static constexpr int state = M * DV * 2;                           // floats
    static constexpr int tokvec = 8 * M + 3 * DV + 4;                  // floats, one set
    static constexpr size_t bytes = (size_t)(2 * state + NW * DV * 4 + 2 * tokvec + 4 * DV + 64) * 4;
};

__device__ __forceinline__ void cp_async16(float *dst_smem, const float *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// N consecutive float2 (N = 1, 2, 4) with the widest accesses; p is aligned to 8 N bytes (16 for N = 4)
template <int N>
__device__ __forceinline__ void ld_row(const float2 *p, float2 (&x)[N])
{
    if constexpr (N == 1) {
        x[0] = *p;
    } else {
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
            const float4 t = reinterpret_cast<const float4 *>(p)[i];
            x[2 * i] = make_float2(t.x, t.y);
            x[2 * i + 1] = make_float2(t.z, t.w);
        }
    }
}
template <int N>
__device__ __forceinline__ void st_row(float2 *p, const float2 (&x)[N])
{
    if constexpr (N == 1) {
        *p = x[0];
    } else {
#pragma unroll
        for (int i = 0; i < N / 2; ++i)
            reinterpret_cast<float4 *>(p)[i] = make_float4(x[2 * i].x, x[2 * i].y, x[2 * i + 1].x, x[2 * i + 1].y);
    }
}

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
    static_assert(DVT % DV == 0, "the value columns split into equal blocks");
    using L = BwdSmem<DK, DV>;
    constexpr int M = L::M, NW = L::NW, TR = L::TR, TC = L::TC;
    static_assert(M + DV + 1 <= kBwdThreads, "one thread per staged value");
    extern __shared__ __align__(16) float sm[];
    float2 *const Sbuf0 = reinterpret_cast<float2 *>(sm);                        // S_{t-1}, two buffers [M][DV]
    float4 *const red = reinterpret_cast<float4 *>(sm + 2 * L::state);           // [NW][DV] partial column sums
    float *const tok0 = sm + 2 * L::state + NW * DV * 4;                         // two sets of token vectors
    float2 *const v_p = reinterpret_cast<float2 *>(tok0 + 2 * L::tokvec);        // p per column (backward)
    float2 *const v_u = v_p + DV;                                                // u (backward) / e = beta u (forward)
    float *const scal = reinterpret_cast<float *>(v_u + DV);                     // [4 w + x]: scalar sums of warp w
    auto Sbuf = [&](int i) { return Sbuf0 + i * (M * DV); };
    // token vectors of set i: per row (lam re, lam im, k re, k im), (q re, q im, cos theta, sin theta); per column
    // yb (re, im) and v; beta
    auto t_lk = [&](int i) { return reinterpret_cast<float4 *>(tok0 + i * L::tokvec); };
    auto t_qc = [&](int i) { return reinterpret_cast<float4 *>(tok0 + i * L::tokvec) + M; };
    auto t_y = [&](int i) { return reinterpret_cast<float2 *>(tok0 + i * L::tokvec + 8 * M); };
    auto t_v = [&](int i) { return tok0 + i * L::tokvec + 8 * M + 2 * DV; };
    auto t_beta = [&](int i) { return tok0 + i * L::tokvec + 8 * M + 3 * DV; };

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bh = blockIdx.x, h = bh % a.H, b = bh / a.H, slice = blockIdx.y, c0 = slice * DV;
    const int T_ = a.T, H = a.H;
    const T *q = static_cast<const T *>(a.q), *k = static_cast<const T *>(a.k), *v = static_cast<const T *>(a.v);
    const T *d_o = static_cast<const T *>(a.d_o), *d_oi = static_cast<const T *>(a.d_o_im);
    float *check = a.check + ((size_t)bh * NSL + slice) * a.NS * 2 * M * DV;
    float *scratch = a.scratch + ((size_t)bh * NSL + slice) * kSeg * 2 * M * DV;
    const int j0 = warp * TR, cl = lane * TC;      // this thread's tile: rows j0 + r, columns cl + x

    // ---- token vectors: global -> registers (issued a step ahead) -> one of the two sets in shared memory
    // (staged by the last M + DV + 1 threads: the first DV are the ones that reduce the column sums meanwhile)
    const int sid = kBwdThreads - 1 - tid;
    float r0 = 0.f, r1 = 0.f, r2 = 0.f, r3 = 0.f, r4 = 0.f, r5 = 0.f;
    auto load_tok = [&](int t, bool back) {
        if (t < 0 || t >= T_) return;
        const size_t row = ((size_t)b * T_ + t) * H + h;
        if (sid < M) {
            r0 = a.alpha[row * M + sid];
            r1 = a.theta[row * M + sid];
            r2 = ld_val(k, row * DK + 2 * sid);
            r3 = ld_val(k, row * DK + 2 * sid + 1);
            if (back) {
                r4 = ld_val(q, row * DK + 2 * sid);
                r5 = ld_val(q, row * DK + 2 * sid + 1);
            }
        } else if (sid < M + DV) {
            const int cc = sid - M;
            r0 = ld_val(v, row * DVT + c0 + cc);
            if (back) {
                r1 = ld_val(d_o, row * DVT + c0 + cc);
                r2 = d_oi ? ld_val(d_oi, row * DVT + c0 + cc) : 0.f;
            }
        } else if (sid == M + DV) {
            r0 = a.beta[row];
        }
    };
    auto stage_tok = [&](int set, bool back) {
        if (sid < M) {
            float sn, cs;
            sincosf(r1, &sn, &cs);
            t_lk(set)[sid] = make_float4(r0 * cs, r0 * sn, r2, r3);
            if (back) t_qc(set)[sid] = make_float4(r4, r5, cs, sn);
        } else if (sid < M + DV) {
            const int cc = sid - M;
            t_v(set)[cc] = r0;
            if (back) t_y(set)[cc] = make_float2(r1, r2);
        } else if (sid == M + DV) {
            t_beta(set)[0] = r0;
        }
    };

    // ---- one forward step on the tile s (registers).  Set `set` holds the token's vectors (visible to all); the
    // next token's vectors, already in registers, are staged into the other set on the way.
    auto fwd_step = [&](float2 (&s)[TR][TC], int set, bool stage_next) {
        const float4 *lkv = t_lk(set);
        float2 kz[TC];
#pragma unroll
        for (int x = 0; x < TC; ++x) kz[x] = make_float2(0.f, 0.f);
#pragma unroll
        for (int r = 0; r < TR; ++r) {
            const float4 lk = lkv[j0 + r];
#pragma unroll
            for (int x = 0; x < TC; ++x) {
                const float zr = lk.x * s[r][x].x - lk.y * s[r][x].y, zi = lk.x * s[r][x].y + lk.y * s[r][x].x;   // Z = Lambda S
                s[r][x] = make_float2(zr, zi);
                kz[x].x += lk.z * zr + lk.w * zi;                                  // conj(k) z
                kz[x].y += lk.z * zi - lk.w * zr;
            }
        }
#pragma unroll
        for (int x = 0; x < TC; ++x) reinterpret_cast<float2 *>(red)[(warp * TC + x) * 32 + lane] = kz[x];
        __syncthreads();
        if (tid < DV) {                     // warp x' of these sums column x' of every lane's tile
            const int c = lane * TC + warp;
            float sr_ = 0.f, si_ = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const float2 x = reinterpret_cast<const float2 *>(red)[(w * TC + warp) * 32 + lane];
                sr_ += x.x;
                si_ += x.y;
            }
            const float bt = t_beta(set)[0];
            v_u[c] = make_float2(bt * (t_v(set)[c] - sr_), -bt * si_);              // e = beta u, u = v - k^* Z
        }
        if (stage_next) stage_tok(set ^ 1, false);
        __syncthreads();
        float2 e[TC];
        ld_row<TC>(v_u + cl, e);
#pragma unroll
        for (int r = 0; r < TR; ++r) {
            const float4 lk = lkv[j0 + r];
#pragma unroll
            for (int x = 0; x < TC; ++x) {
                s[r][x].x += lk.z * e[x].x - lk.w * e[x].y;
                s[r][x].y += lk.z * e[x].y + lk.w * e[x].x;
            }
        }
    };

    // ---- a tile between registers and global memory (workspace format: interleaved complex [M][DV])
    auto store_tile = [&](const float2 (&s)[TR][TC], float *dst) {
#pragma unroll
        for (int r = 0; r < TR; ++r) st_row<TC>(reinterpret_cast<float2 *>(dst) + (size_t)(j0 + r) * DV + cl, s[r]);
    };
    auto load_tile = [&](float2 (&s)[TR][TC], const float *src) {
#pragma unroll
        for (int r = 0; r < TR; ++r) ld_row<TC>(reinterpret_cast<const float2 *>(src) + (size_t)(j0 + r) * DV + cl, s[r]);
    };
    auto load_state_async = [&](float2 *S, const float *src) {
        for (int idx = tid; idx < M * DV / 2; idx += kBwdThreads) cp_async16(reinterpret_cast<float *>(S) + 4 * idx, src + 4 * idx);
        cp_async_commit();
    };

    // ---- sweep 1: forward, checkpoints at the start of every segment (nothing is needed beyond the last one)
    float2 s[TR][TC];
#pragma unroll
    for (int r = 0; r < TR; ++r)
#pragma unroll
        for (int x = 0; x < TC; ++x) {
            const size_t at = ((size_t)bh * DK + 2 * (j0 + r)) * DVT + c0 + cl + x;
            s[r][x] = a.S0 ? make_float2(a.S0[at], a.S0[at + DVT]) : make_float2(0.f, 0.f);
        }
    const int t_last_check = (a.NS - 1) * kSeg;
    int set = 0;
    load_tok(0, false);
    stage_tok(set, false);
    __syncthreads();
    for (int t = 0; t < t_last_check; ++t) {
        if (t % kSeg == 0) store_tile(s, check + (size_t)(t / kSeg) * 2 * M * DV);
        load_tok(t + 1, false);
        fwd_step(s, set, true);
        set ^= 1;
    }
    store_tile(s, check + (size_t)(a.NS - 1) * 2 * M * DV);

    // ---- cotangent of the final state
    float2 G[TR][TC];
#pragma unroll
    for (int r = 0; r < TR; ++r)
#pragma unroll
        for (int x = 0; x < TC; ++x) {
            const size_t at = ((size_t)bh * DK + 2 * (j0 + r)) * DVT + c0 + cl + x;
            G[r][x] = a.dS_T ? make_float2(a.dS_T[at], a.dS_T[at + DVT]) : make_float2(0.f, 0.f);
        }

    T *dq = static_cast<T *>(a.dq), *dk = static_cast<T *>(a.dk), *dv = static_cast<T *>(a.dv);
    float *dq_p = a.dq_p + (size_t)slice * a.rows * DK, *dk_p = a.dk_p + (size_t)slice * a.rows * DK;
    float *dal_p = a.dalpha_p + (size_t)slice * a.rows * M, *dth_p = a.dtheta_p + (size_t)slice * a.rows * M;
    float *dbe_p = a.dbeta_p + (size_t)slice * a.rows;
    for (int si = a.NS - 1; si >= 0; --si) {
        const int t0 = si * kSeg, t1 = min(t0 + kSeg, T_);
        // ---- sweep 2: forward again from the checkpoint (this thread wrote the tile it reads), S_{t-1} of every
        // token to the scratch
        __syncthreads();                  // every reader of the token vectors and of v_u is done
        load_tile(s, check + (size_t)si * 2 * M * DV);
        set = 0;
        load_tok(t0, false);
        stage_tok(set, false);
        __syncthreads();
        for (int t = t0; t < t1; ++t) {
            store_tile(s, scratch + (size_t)(t - t0) * 2 * M * DV);
            if (t + 1 < t1) {                                   // the state after the last token is not needed
                load_tok(t + 1, false);
                fwd_step(s, set, true);
                set ^= 1;
            }
        }
        __syncthreads();      // the scratch stores of this CTA are visible to its own later loads

        // ---- sweep 3: backward through the segment; S_{t-1} arrives one token ahead in the other buffer
        int buf = 0;
        set = 0;
        load_state_async(Sbuf(buf), scratch + (size_t)(t1 - 1 - t0) * 2 * M * DV);
        load_tok(t1 - 1, true);
        stage_tok(set, true);
        cp_async_wait_all();
        __syncthreads();
        for (int t = t1 - 1; t >= t0; --t) {
            if (t > t0) {
                load_state_async(Sbuf(buf ^ 1), scratch + (size_t)(t - 1 - t0) * 2 * M * DV);
                load_tok(t - 1, true);
            }
            const float4 *lkv = t_lk(set), *qcv = t_qc(set);
            const float bt = t_beta(set)[0];
            const size_t row = ((size_t)b * T_ + t) * H + h;
            float2 y[TC];
            ld_row<TC>(t_y(set) + cl, y);

            // step 1: G += q yb^*; partial sums over this warp's rows of p = G^* k and k^* Z
            {
                float4 acc[TC];
#pragma unroll
                for (int x = 0; x < TC; ++x) acc[x] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int r = 0; r < TR; ++r) {
                    const float4 lk = lkv[j0 + r], qc = qcv[j0 + r];
                    ld_row<TC>(Sbuf(buf) + (j0 + r) * DV + cl, s[r]);
#pragma unroll
                    for (int x = 0; x < TC; ++x) {
                        const float gr = G[r][x].x + qc.x * y[x].x + qc.y * y[x].y;          // G + q conj(yb)
                        const float gi = G[r][x].y + qc.y * y[x].x - qc.x * y[x].y;
                        G[r][x] = make_float2(gr, gi);
                        acc[x].x += gr * lk.z + gi * lk.w;                                  // conj(G) k
                        acc[x].y += gr * lk.w - gi * lk.z;
                        const float zr = lk.x * s[r][x].x - lk.y * s[r][x].y, zi = lk.x * s[r][x].y + lk.y * s[r][x].x;
                        acc[x].z += lk.z * zr + lk.w * zi;                                  // conj(k) z
                        acc[x].w += lk.z * zi - lk.w * zr;
                    }
                }
#pragma unroll
                for (int x = 0; x < TC; ++x) red[(warp * TC + x) * 32 + lane] = acc[x];     // [warp][x][lane]: no bank conflicts
            }
            __syncthreads();
            // step 2: p, u per column; dv; the sums over columns u^T p and u^T yb (one set per warp of columns)
            if (tid < DV) {                 // warp x' of these sums column x' of every lane's tile
                const int c = lane * TC + warp;
                float pr = 0.f, pi = 0.f, zr = 0.f, zi = 0.f;
#pragma unroll
                for (int w = 0; w < NW; ++w) {
                    const float4 x = red[(w * TC + warp) * 32 + lane];
                    pr += x.x;  pi += x.y;  zr += x.z;  zi += x.w;
                }
                const float ur = t_v(set)[c] - zr, ui = -zi;
                const float2 yy = t_y(set)[c];
                v_p[c] = make_float2(pr, pi);
                v_u[c] = make_float2(ur, ui);
                st_val(dv, row * DVT + c0 + c, bt * pr);
                float s0 = ur * pr - ui * pi;                                   // Re(u p)
                float s1 = ur * yy.x - ui * yy.y, s2 = ur * yy.y + ui * yy.x;   // u yb
#pragma unroll
                for (int d = 16; d >= 1; d >>= 1) {
                    s0 += __shfl_xor_sync(0xffffffffu, s0, d);
                    s1 += __shfl_xor_sync(0xffffffffu, s1, d);
                    s2 += __shfl_xor_sync(0xffffffffu, s2, d);
                }
                if (lane == 0) { scal[4 * warp] = s0; scal[4 * warp + 1] = s1; scal[4 * warp + 2] = s2; }
            }
            if (t > t0) stage_tok(set ^ 1, true);
            cp_async_wait_all();
            __syncthreads();
            // step 3: this warp's rows: shares of dq, dk, dalpha, dtheta; G <- conj(lam) (G - beta k p^*)
            {
                float uy_r = 0.f, uy_i = 0.f, dbe = 0.f;
#pragma unroll
                for (int w = 0; w < DV / 32; ++w) { dbe += scal[4 * w]; uy_r += scal[4 * w + 1]; uy_i += scal[4 * w + 2]; }
                if (tid == 0) (NSL == 1 ? a.dbeta : dbe_p)[row] = dbe;
                float2 pp[TC], uu[TC];
                ld_row<TC>(v_p + cl, pp);
                ld_row<TC>(v_u + cl, uu);
                // per row: dq re, im; dk re, im (before the factor beta); dalpha; dtheta; two unused
                constexpr int NV = 8 * TR;
                float val[NV];
#pragma unroll
                for (int r = 0; r < TR; ++r) {
                    const float4 lk = lkv[j0 + r], qc = qcv[j0 + r];
                    const float lr = lk.x, li = lk.y, kr = lk.z, ki = lk.w;
                    float qzr = 0.f, qzi = 0.f, dkr = 0.f, dki = 0.f, lbr = 0.f, lbi = 0.f;
#pragma unroll
                    for (int x = 0; x < TC; ++x) {
                        const float gr = G[r][x].x, gi = G[r][x].y, sr = s[r][x].x, si2 = s[r][x].y;
                        const float yr = y[x].x, yi = y[x].y, ur = uu[x].x, ui = uu[x].y, pr = pp[x].x, pi = pp[x].y;
                        const float zr = lr * sr - li * si2, zi = lr * si2 + li * sr;
                        qzr += zr * yr - zi * yi;  qzi += zr * yi + zi * yr;                 // Z yb
                        dkr += gr * ur + gi * ui - (zr * pr - zi * pi);                      // G conj(u) - Z p
                        dki += gi * ur - gr * ui - (zr * pi + zi * pr);
                        // Zb = G - beta k conj(p)
                        const float br = gr - bt * (kr * pr + ki * pi), bi = gi - bt * (ki * pr - kr * pi);
                        lbr += sr * br + si2 * bi;  lbi += sr * bi - si2 * br;               // conj(S_{t-1}) Zb
                        G[r][x] = make_float2(lr * br + li * bi, lr * bi - li * br);         // conj(lam) Zb
                    }
                    val[8 * r + 0] = qzr;
                    val[8 * r + 1] = qzi;
                    val[8 * r + 2] = bt * dkr;
                    val[8 * r + 3] = bt * dki;
                    val[8 * r + 4] = lbr * qc.z + lbi * qc.w;                                // Re(conj(lamb) e^{i theta})
                    val[8 * r + 5] = lbi * lr - lbr * li;                                    // -Im(conj(lamb) lam)
                    val[8 * r + 6] = 0.f;
                    val[8 * r + 7] = 0.f;
                }
                // sums over the warp's lanes (= columns): every exchange halves the values a lane still carries, so
                // that lane l ends with the total of value l (NV = 32) or l / 2 (NV = 16)
                int n = NV;
#pragma unroll
                for (int d = 16; d >= 1; d >>= 1) {
                    if (n > 1) {
                        const int half = n / 2;
                        const bool up = (lane & d) != 0;
#pragma unroll
                        for (int i = 0; i < NV / 2; ++i) {
                            if (i < half) {
                                const float send = up ? val[i] : val[i + half];
                                const float keep = up ? val[i + half] : val[i];
                                val[i] = keep + __shfl_xor_sync(0xffffffffu, send, d);
                            }
                        }
                        n = half;
                    } else {
                        val[0] += __shfl_xor_sync(0xffffffffu, val[0], d);
                    }
                }
                const int vi = NV == 32 ? lane : lane >> 1;
                const int rr = vi >> 3, qq = vi & 7, j = j0 + rr;
                if (qq < 6 && (NV == 32 || !(lane & 1))) {
                    float out = val[0];
                    if (qq < 2) {
                        const float4 lk = lkv[j];
                        out += qq == 0 ? bt * (lk.z * uy_r - lk.w * uy_i) : bt * (lk.z * uy_i + lk.w * uy_r);   // + beta k (u^T yb)
                    }
                    if constexpr (NSL == 1) {
                        if (qq < 2) st_val(dq, row * DK + 2 * j + qq, out);
                        else if (qq < 4) st_val(dk, row * DK + 2 * j + qq - 2, out);
                        else if (qq == 4) a.dalpha[row * M + j] = out;
                        else a.dtheta[row * M + j] = out;
                    } else {      // this column block's share of the sums over the columns
                        if (qq < 2) dq_p[row * DK + 2 * j + qq] = out;
                        else if (qq < 4) dk_p[row * DK + 2 * j + qq - 2] = out;
                        else if (qq == 4) dal_p[row * M + j] = out;
                        else dth_p[row * M + j] = out;
                    }
                }
            }
            buf ^= 1;
            set ^= 1;
        }
    }
#pragma unroll
    for (int r = 0; r < TR; ++r)
#pragma unroll
        for (int x = 0; x < TC; ++x) {
            const size_t at = ((size_t)bh * DK + 2 * (j0 + r)) * DVT + c0 + cl + x;
            a.dS0[at] = G[r][x].x;
            a.dS0[at + DVT] = G[r][x].y;
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
