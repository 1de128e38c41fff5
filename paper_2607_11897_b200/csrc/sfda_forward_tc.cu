// Tensor-core chunk-WY forward for sm_100a: bf16 q/k/v, d_k = d_v = 128, chunk C = 64.
//
// One CTA walks the chunks of one (batch, head) pair.  The fp32 state lives in tensor memory for the
// whole sequence, transposed: TMEM lane c = value channel, column = key channel in de-interleaved order
// [Re j = 0..63 | Im j = 0..63].  Every dense contraction is a tcgen05.mma (kind::f16, bf16 operands,
// fp32 accumulators in TMEM); the state-dependent ones take their A operand (bf16 copies of S, R, E) from
// TMEM and their B operand from 128-byte-swizzled K-major shared-memory tiles that the CUDA cores build.
//
// With gamma_t = a_t e^{i phi_t} the chunk-local cumulative phase-decay (Eq. "constructive-Gamma"),
// k'_t = e^{-i phi_t} k_t, q'_t = e^{-i phi_t} q_t:
//
//   W_t   = a_t k'_t                (= conj(gamma_t) k_t, Eq. "constructive-W")
//   Kc_t  = k'_t / a_t              (= k_t / gamma_t)
//   Qt_t  = a_t q'_t                (= conj(gamma_t) q_t)
//   Y'_t  = (a_C / a_t) k'_t        (= e^{-i phi_C} (gamma_C / gamma_t) k_t, cf. Eq. "constructive-Y")
//   Kt[t][i] = W_t^* Kc_i (i < t),  Aq[t][i] = Qt_t^* Kc_i (i <= t)          -- Gram blocks
//   M_beta = (I + D_beta Kt)^{-1} D_beta                                     -- unit-lower WY system
//   R = V - W^* S_0,  E = M_beta R                                           -- Eq. "apply-transfer"
//   rho_t = Qt_t^* S_0 + sum_{i<=t} Aq[t][i] e_i^T,  o_t = conj(rho_t)       -- Thm "Prefix outputs"
//   S_C = e^{i phi_C} (a_C S_0 + sum_t Y'_t e_t^T)                           -- boundary-state scan
//
// Complex products are real block products over the de-interleaved halves; where a minus sign is needed
// the instruction descriptor's negate-B bit supplies it, so no operand is stored twice.
#include <cuda.h>

#include "sfda_common.cuh"
#include "sfda_internal.h"
#include "sfda_tc_ptx.cuh"

namespace sfda {
namespace {

using namespace tc;

constexpr int C = 64;         // chunk
constexpr int DK = 128, DV = 128, M = 64;
constexpr int kThreads = 256;

// ---- shared memory map (bytes from a 1024-aligned base) -------------------------------------------
constexpr int kTile = 8192;                      // 64 rows x 128 B, K-major, 128B swizzle
constexpr int OFF_WQ_RE = 0;                     // 128 rows: W (0..63) then Qt (64..127), Re halves
constexpr int OFF_WQ_IM = OFF_WQ_RE + 2 * kTile;
constexpr int OFF_KC_RE = OFF_WQ_IM + 2 * kTile;
constexpr int OFF_KC_IM = OFF_KC_RE + kTile;
constexpr int OFF_YT_RE = OFF_KC_IM + kTile;     // Y'^T [j][t]
constexpr int OFF_YT_IM = OFF_YT_RE + kTile;
constexpr int OFF_MB_RE = OFF_YT_IM + kTile;     // M_beta [t][i]
constexpr int OFF_MB_IM = OFF_MB_RE + kTile;
constexpr int OFF_AQ_RE = OFF_MB_IM + kTile;     // Aq [t][i], upper triangle zero
constexpr int OFF_AQ_IM = OFF_AQ_RE + kTile;
constexpr int OFF_V = OFF_AQ_IM + kTile;         // v staging [t][128] bf16 (TMA, no swizzle)
constexpr int OFF_Q = OFF_V + 16384;             // q staging [t][128] bf16
constexpr int OFF_K = OFF_Q + 16384;             // k staging
constexpr int OFF_ALPHA = OFF_K + 16384;         // alpha staging [t][64] fp32
constexpr int OFF_THETA = OFF_ALPHA + 16384;     // theta staging
constexpr int OFF_SOLVE = OFF_Q;                 // L, X (fp32 complex 64 x 64, row stride 68) alias the staging
constexpr int LS = 68;                           // row stride (floats) of L and X: conflict-free A fragments
constexpr int TS = 40;                           // row stride of the T scratch: conflict-free B fragments
constexpr int OFF_MISC = OFF_SOLVE + 4 * 64 * LS * 4;
constexpr int kSmemBytes = OFF_MISC + 20480 + 1024;   // + slack for the 1024-byte alignment
static_assert(OFF_MISC >= OFF_THETA + 16384, "solve scratch must cover the staging buffers it aliases");

struct Misc {
    float part_lg[8][M];
    uint32_t part_turns[8][M];
    float aC[M];
    float closing_cos[2][M], closing_sin[2][M];
    float beta[C];
    float Tr[32 * TS], Ti[32 * TS];
    unsigned long long bar_mma, bar_in, bar_v;
    uint32_t tmem_base;
};
static_assert(sizeof(Misc) <= 20480, "misc area too small");

// ---- tensor memory map (columns) -------------------------------------------------------------------
constexpr uint32_t TM_S32 = 0;     // state fp32: [Re j | Im j]
constexpr uint32_t TM_S16 = 128;   // bf16 copy of the chunk-start state (A operand), 64 packed columns
constexpr uint32_t TM_X16 = 192;   // bf16 R, then E (A operand)
constexpr uint32_t TM_ACC = 256;   // [D1/E re | rho re | D1/E im | rho im], 64 columns each; Gram uses 0..127

// Optional per-phase cycle counters (development builds only, -DSFDA_TC_TIMING).
#ifdef SFDA_TC_TIMING
#define SFDA_MARK(i)                                                          \
    do {                                                                      \
        if (tid == 0 && bh == 0 && p.timing) {                                \
            const long long now_ = clock64();                                 \
            p.timing[i] += now_ - mark_;                                      \
            mark_ = now_;                                                     \
        }                                                                     \
    } while (0)
#else
#define SFDA_MARK(i) \
    do {             \
    } while (0)
#endif

struct Params {
#ifdef SFDA_TC_TIMING
    long long *timing;
#endif
    const float *beta, *S0;
    __nv_bfloat16 *o, *o_im;
    float *S_T;
    uint32_t *status;
    int T, H;
};

// ---- the kernel -------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1)
sfda_forward_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_alpha,
                       const __grid_constant__ CUtensorMap tm_theta, const __grid_constant__ CUtensorMap tm_o,
                       const __grid_constant__ CUtensorMap tm_oim, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Misc &mi = *reinterpret_cast<Misc *>(smem + OFF_MISC);
    float *Lr = reinterpret_cast<float *>(smem + OFF_SOLVE);
    float *Li = Lr + 64 * LS, *Xr = Li + 64 * LS, *Xi = Xr + 64 * LS;
    const uint32_t sbase = smem_u32(smem);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int quad = warp & 3, half = warp >> 2;
    const int bh = blockIdx.x, h = bh % p.H, b = bh / p.H;
    const int n_chunks = (p.T + C - 1) / C;

    if (tid == 0) {
        mbar_init(&mi.bar_mma, 1);
        mbar_init(&mi.bar_in, 1);
        mbar_init(&mi.bar_v, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&mi.tmem_base)));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = mi.tmem_base;
    const uint32_t tlane = tmem + ((uint32_t)(quad * 32) << 16);   // this warp's lane quadrant

    if (tid == 0) {
        mbar_expect_tx(&mi.bar_in, 4 * 16384);
        tma_load_4d(smem + OFF_Q, &tm_q, &mi.bar_in, 0, h, 0, b);
        tma_load_4d(smem + OFF_K, &tm_k, &mi.bar_in, 0, h, 0, b);
        tma_load_4d(smem + OFF_ALPHA, &tm_alpha, &mi.bar_in, 0, h, 0, b);
        tma_load_4d(smem + OFF_THETA, &tm_theta, &mi.bar_in, 0, h, 0, b);
        mbar_expect_tx(&mi.bar_v, 16384);
        tma_load_4d(smem + OFF_V, &tm_v, &mi.bar_v, 0, h, 0, b);
    }

#ifdef SFDA_TC_TIMING
    long long mark_ = clock64();
#endif
    uint32_t ph_mma = 0, ph_in = 0, ph_v = 0;
    bool in_flight_in = true, in_flight_v = true;
    int failed = 0;

    for (int ci = 0; ci < n_chunks; ++ci) {
        const int t0 = ci * C;
        const int len = min(C, p.T - t0);
        const int cur = ci & 1;

        // ================= prep: cumulative phase-decay and the operand tiles =======================
        if (tid == 0) tma_store_wait_read();   // the previous chunk's output store still reads the WQ tiles
        failed = __syncthreads_or(mbar_wait(&mi.bar_in, ph_in) ? 0 : 1);
        ph_in ^= 1;
        in_flight_in = false;
        if (failed) break;
        SFDA_MARK(0);
        {
            // thread = (channel pair jp: channels 2jp, 2jp+1 ; token octet tq = warp)
            const int jp = tid & 31, tq = tid >> 5;
            const float2 *s_alpha = reinterpret_cast<const float2 *>(smem + OFF_ALPHA);
            const float2 *s_theta = reinterpret_cast<const float2 *>(smem + OFF_THETA);
            float lg0[8], lg1[8];
            uint32_t tu0[8], tu1[8];
            float acc0 = 0.f, acc1 = 0.f;
            uint32_t tacc0 = 0u, tacc1 = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int t = tq * 8 + i;
                if (t < len) {
                    const float2 al = s_alpha[t * 32 + jp], th = s_theta[t * 32 + jp];
                    acc0 += fmaxf(__log2f(al.x), -43.28f);   // floor e^-30, as in log_decay
                    acc1 += fmaxf(__log2f(al.y), -43.28f);
                    tacc0 += phase_to_turns(th.x);
                    tacc1 += phase_to_turns(th.y);
                }
                lg0[i] = acc0; lg1[i] = acc1;
                tu0[i] = tacc0; tu1[i] = tacc1;
            }
            mi.part_lg[tq][2 * jp] = acc0;
            mi.part_lg[tq][2 * jp + 1] = acc1;
            mi.part_turns[tq][2 * jp] = tacc0;
            mi.part_turns[tq][2 * jp + 1] = tacc1;
            if (tid < C) mi.beta[tid] = tid < len ? p.beta[((size_t)b * p.T + t0 + tid) * p.H + h] : 0.f;
            __syncthreads();
            float base0 = 0.f, base1 = 0.f, tot0 = 0.f, tot1 = 0.f;
            uint32_t tb0 = 0u, tb1 = 0u, tt0 = 0u, tt1 = 0u;
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                const float2 pl = *reinterpret_cast<const float2 *>(&mi.part_lg[g][2 * jp]);
                const uint2 pt = *reinterpret_cast<const uint2 *>(&mi.part_turns[g][2 * jp]);
                if (g < tq) { base0 += pl.x; base1 += pl.y; tb0 += pt.x; tb1 += pt.y; }
                tot0 += pl.x; tot1 += pl.y; tt0 += pt.x; tt1 += pt.y;
            }
            if (tq == 0) {
                float cs, sn;
                mi.aC[2 * jp] = exp2f(tot0);
                mi.aC[2 * jp + 1] = exp2f(tot1);
                __sincosf((float)(int32_t)tt0 * 0x1.921fb6p-30f, &sn, &cs);   // turns * 2 pi / 2^32
                mi.closing_cos[cur][2 * jp] = cs;
                mi.closing_sin[cur][2 * jp] = sn;
                __sincosf((float)(int32_t)tt1 * 0x1.921fb6p-30f, &sn, &cs);
                mi.closing_cos[cur][2 * jp + 1] = cs;
                mi.closing_sin[cur][2 * jp + 1] = sn;
            }
            const uint2 *s_q = reinterpret_cast<const uint2 *>(smem + OFF_Q);
            const uint2 *s_k = reinterpret_cast<const uint2 *>(smem + OFF_K);
            uint32_t y0r[4], y0i[4], y1r[4], y1i[4];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int t = tq * 8 + i;
                const uint2 kw = s_k[t * 32 + jp], qw = s_q[t * 32 + jp];
                float wr[2], wi[2], cr_[2], ci_[2], qr_[2], qi_[2], yr[2], yi[2];
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    const float l2 = x ? base1 + lg1[i] : base0 + lg0[i];
                    const float tot = x ? tot1 : tot0;
                    const uint32_t tu = x ? tb1 + tu1[i] : tb0 + tu0[i];
                    const uint32_t kx = x ? kw.y : kw.x, qx = x ? qw.y : qw.x;
                    const float a = exp2f(l2);
                    const float ainv = exp2f(fminf(-l2, 115.4f));                 // 1/a_t, capped at e^80
                    const float ay = exp2f(tot - l2);                             // a_C / a_t <= 1
                    float cs, sn;
                    __sincosf((float)(int32_t)tu * 0x1.921fb6p-30f, &sn, &cs);
                    const float kr = __uint_as_float(kx << 16), ki = __uint_as_float(kx & 0xffff0000u);
                    const float qr = __uint_as_float(qx << 16), qi = __uint_as_float(qx & 0xffff0000u);
                    const float kpr = kr * cs + ki * sn, kpi = ki * cs - kr * sn;   // e^{-i phi} k
                    const float qpr = qr * cs + qi * sn, qpi = qi * cs - qr * sn;
                    wr[x] = a * kpr; wi[x] = a * kpi;
                    qr_[x] = a * qpr; qi_[x] = a * qpi;
                    cr_[x] = ainv * kpr; ci_[x] = ainv * kpi;
                    yr[x] = ay * kpr; yi[x] = ay * kpi;
                }
                const int o1 = sw_off(t, 2 * jp);
                *reinterpret_cast<uint32_t *>(smem + OFF_WQ_RE + o1) = pack_bf16(wr[0], wr[1]);
                *reinterpret_cast<uint32_t *>(smem + OFF_WQ_IM + o1) = pack_bf16(wi[0], wi[1]);
                *reinterpret_cast<uint32_t *>(smem + OFF_WQ_RE + kTile + o1) = pack_bf16(qr_[0], qr_[1]);
                *reinterpret_cast<uint32_t *>(smem + OFF_WQ_IM + kTile + o1) = pack_bf16(qi_[0], qi_[1]);
                *reinterpret_cast<uint32_t *>(smem + OFF_KC_RE + o1) = pack_bf16(cr_[0], cr_[1]);
                *reinterpret_cast<uint32_t *>(smem + OFF_KC_IM + o1) = pack_bf16(ci_[0], ci_[1]);
                const uint32_t h0r = __bfloat16_as_ushort(__float2bfloat16_rn(yr[0]));
                const uint32_t h0i = __bfloat16_as_ushort(__float2bfloat16_rn(yi[0]));
                const uint32_t h1r = __bfloat16_as_ushort(__float2bfloat16_rn(yr[1]));
                const uint32_t h1i = __bfloat16_as_ushort(__float2bfloat16_rn(yi[1]));
                if (i & 1) {
                    y0r[i >> 1] |= h0r << 16; y0i[i >> 1] |= h0i << 16;
                    y1r[i >> 1] |= h1r << 16; y1i[i >> 1] |= h1i << 16;
                } else {
                    y0r[i >> 1] = h0r; y0i[i >> 1] = h0i;
                    y1r[i >> 1] = h1r; y1i[i >> 1] = h1i;
                }
            }
            // Y'^T rows 2jp and 2jp+1, tokens 8 tq .. 8 tq + 7: one 16-byte chunk per row and half.
            const int oa = sw_off(2 * jp, tq * 8), ob = sw_off(2 * jp + 1, tq * 8);
            *reinterpret_cast<uint4 *>(smem + OFF_YT_RE + oa) = make_uint4(y0r[0], y0r[1], y0r[2], y0r[3]);
            *reinterpret_cast<uint4 *>(smem + OFF_YT_IM + oa) = make_uint4(y0i[0], y0i[1], y0i[2], y0i[3]);
            *reinterpret_cast<uint4 *>(smem + OFF_YT_RE + ob) = make_uint4(y1r[0], y1r[1], y1r[2], y1r[3]);
            *reinterpret_cast<uint4 *>(smem + OFF_YT_IM + ob) = make_uint4(y1i[0], y1i[1], y1i[2], y1i[3]);
        }
        fence_async_smem();
        tc_fence_before();
        __syncthreads();

        SFDA_MARK(1);
        // ================= Gram blocks Kt (rows 0..63) and Aq (rows 64..127) ==========================
        if (tid == 0) {
            tc_fence_after();
            const uint32_t d_re = tmem + TM_ACC, d_im = tmem + TM_ACC + 64;
            mma_k64_ss(d_re, sbase + OFF_WQ_RE, sbase + OFF_KC_RE, idesc(64, 0), false);
            mma_k64_ss(d_re, sbase + OFF_WQ_IM, sbase + OFF_KC_IM, idesc(64, 0), true);
            mma_k64_ss(d_im, sbase + OFF_WQ_RE, sbase + OFF_KC_IM, idesc(64, 0), false);
            mma_k64_ss(d_im, sbase + OFF_WQ_IM, sbase + OFF_KC_RE, idesc(64, 1), true);
            mma_commit(&mi.bar_mma);
        }
        failed = __syncthreads_or(mbar_wait(&mi.bar_mma, ph_mma) ? 0 : 1);
        ph_mma ^= 1;
        if (failed) break;
        tc_fence_after();
        SFDA_MARK(2);
        {
            uint32_t r[64];
            tmem_ld<64>(tlane + TM_ACC + 64 * half, r);
            tc_wait_ld();
            const int row = quad * 32 + lane;
            if (row < 64) {                       // L = D_beta Kt, strictly lower
                const int t = row;
                const float bt = mi.beta[t];
                float4 *dst = reinterpret_cast<float4 *>((half ? Li : Lr) + t * LS);
#pragma unroll
                for (int i = 0; i < 64; i += 4)
                    dst[i >> 2] = make_float4(i < t ? bt * __uint_as_float(r[i]) : 0.f,
                                              i + 1 < t ? bt * __uint_as_float(r[i + 1]) : 0.f,
                                              i + 2 < t ? bt * __uint_as_float(r[i + 2]) : 0.f,
                                              i + 3 < t ? bt * __uint_as_float(r[i + 3]) : 0.f);
            } else {                              // Aq, lower incl. diagonal, as a bf16 operand tile
                const int t = row - 64;
                uint8_t *tile = smem + (half ? OFF_AQ_IM : OFF_AQ_RE);
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) {
                    uint32_t w[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const int i0 = c8 * 8 + 2 * x;
                        w[x] = pack_bf16(i0 <= t ? __uint_as_float(r[i0]) : 0.f,
                                         i0 + 1 <= t ? __uint_as_float(r[i0 + 1]) : 0.f);
                    }
                    *reinterpret_cast<uint4 *>(tile + sw_off(t, c8 * 8)) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
        tc_fence_before();
        __syncthreads();

        SFDA_MARK(3);
        // ================= X = (I + L)^{-1}: 16x16 diagonal blocks by substitution, merges on mma.sync ===
        if (warp < 4 && lane < 16) {                  // warp b inverts diagonal block b, lane = column
            const int o = 16 * warp, c = lane;
            float xr[16], xi[16];
#pragma unroll
            for (int r = 0; r < 16; ++r) {
                float ar = r == c ? 1.f : 0.f, ai = 0.f;
#pragma unroll
                for (int i = 0; i < 15; ++i) {
                    if (i < r) {
                        const float lr_ = Lr[(o + r) * LS + o + i], li_ = Li[(o + r) * LS + o + i];
                        const float vr = i >= c ? xr[i] : 0.f, vi = i >= c ? xi[i] : 0.f;
                        ar -= lr_ * vr - li_ * vi;
                        ai -= lr_ * vi + li_ * vr;
                    }
                }
                xr[r] = r >= c ? ar : 0.f;
                xi[r] = r >= c ? ai : 0.f;
                Xr[(o + r) * LS + o + c] = xr[r];
                Xi[(o + r) * LS + o + c] = xi[r];
            }
        }
        __syncthreads();
        if (warp < 2) {                               // level 1: X[b1][b0] = -X[b1][b1] (L[b1][b0] X[b0][b0])
            const int r0 = 32 * warp + 16, c0 = 32 * warp;
            float *tr = mi.Tr + 16 * warp * TS, *ti = mi.Ti + 16 * warp * TS;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                float cr[4] = {0.f, 0.f, 0.f, 0.f}, ci[4] = {0.f, 0.f, 0.f, 0.f};
                cmma_16x8(cr, ci, Lr, Li, LS, r0, c0, Xr, Xi, LS, c0, c0 + 8 * nt, nt, 2, lane);
                store_tile(cr, ci, 1.f, tr, ti, TS, 0, 8 * nt, lane);
            }
            __syncwarp();
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                float cr[4] = {0.f, 0.f, 0.f, 0.f}, ci[4] = {0.f, 0.f, 0.f, 0.f};
                cmma_16x8(cr, ci, Xr, Xi, LS, r0, r0, tr, ti, TS, 0, 8 * nt, 0, 2, lane);
                store_tile(cr, ci, -1.f, Xr, Xi, LS, r0, c0 + 8 * nt, lane);
            }
        }
        __syncthreads();
        {                                             // level 2: X[BL] = -X[BR] (L[BL] X[TL]); one tile per warp
            const int mt = warp >> 2, nt = warp & 3;
            float cr[4] = {0.f, 0.f, 0.f, 0.f}, ci[4] = {0.f, 0.f, 0.f, 0.f};
            cmma_16x8(cr, ci, Lr, Li, LS, 32 + 16 * mt, 0, Xr, Xi, LS, 0, 8 * nt, nt, 4, lane);
            store_tile(cr, ci, 1.f, mi.Tr, mi.Ti, TS, 16 * mt, 8 * nt, lane);
            __syncthreads();
            float dr[4] = {0.f, 0.f, 0.f, 0.f}, di[4] = {0.f, 0.f, 0.f, 0.f};
            cmma_16x8(dr, di, Xr, Xi, LS, 32 + 16 * mt, 32, mi.Tr, mi.Ti, TS, 0, 8 * nt, 0, 2 * mt + 2, lane);
            store_tile(dr, di, -1.f, Xr, Xi, LS, 32 + 16 * mt, 8 * nt, lane);
        }
        __syncthreads();
        {
            const int t = tid >> 2, part = tid & 3;     // row t, columns 16 part .. 16 part + 15
#pragma unroll
            for (int cidx = 0; cidx < 2; ++cidx) {
                uint32_t wr[4], wi[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    const int i0 = part * 16 + cidx * 8 + 2 * x;
                    const float b0 = mi.beta[i0], b1 = mi.beta[i0 + 1];
                    const bool in0 = i0 <= t, in1 = i0 + 1 <= t;
                    wr[x] = pack_bf16(in0 ? Xr[t * LS + i0] * b0 : 0.f, in1 ? Xr[t * LS + i0 + 1] * b1 : 0.f);
                    wi[x] = pack_bf16(in0 ? Xi[t * LS + i0] * b0 : 0.f, in1 ? Xi[t * LS + i0 + 1] * b1 : 0.f);
                }
                const int off = sw_off(t, part * 16 + cidx * 8);
                *reinterpret_cast<uint4 *>(smem + OFF_MB_RE + off) = make_uint4(wr[0], wr[1], wr[2], wr[3]);
                *reinterpret_cast<uint4 *>(smem + OFF_MB_IM + off) = make_uint4(wi[0], wi[1], wi[2], wi[3]);
            }
        }

        SFDA_MARK(4);
        // ================= state pass: S16 <- bf16(S_start), S32 <- a_C * S_start ======================
        {
            const int c = quad * 32 + lane;        // value channel = TMEM lane
            const int j0 = half * 32;              // this warp's complex rows
            uint32_t sre[32], sim[32];
            if (ci == 0) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int j = j0 + i;
                    sre[i] = p.S0 ? __float_as_uint(p.S0[((size_t)bh * DK + 2 * j) * DV + c]) : 0u;
                    sim[i] = p.S0 ? __float_as_uint(p.S0[((size_t)bh * DK + 2 * j + 1) * DV + c]) : 0u;
                }
            } else {
                tmem_ld<32>(tlane + TM_S32 + j0, sre);
                tmem_ld<32>(tlane + TM_S32 + 64 + j0, sim);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) {     // closing phase of the previous chunk
                    const float cs = mi.closing_cos[cur ^ 1][j0 + i], sn = mi.closing_sin[cur ^ 1][j0 + i];
                    const float xr = __uint_as_float(sre[i]), xi = __uint_as_float(sim[i]);
                    sre[i] = __float_as_uint(cs * xr - sn * xi);
                    sim[i] = __float_as_uint(cs * xi + sn * xr);
                }
            }
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(__uint_as_float(sre[2 * i]), __uint_as_float(sre[2 * i + 1]));
            tmem_st<16>(tlane + TM_S16 + j0 / 2, pk);
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(__uint_as_float(sim[2 * i]), __uint_as_float(sim[2 * i + 1]));
            tmem_st<16>(tlane + TM_S16 + 32 + j0 / 2, pk);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float a = mi.aC[j0 + i];
                sre[i] = __float_as_uint(a * __uint_as_float(sre[i]));
                sim[i] = __float_as_uint(a * __uint_as_float(sim[i]));
            }
            tmem_st<32>(tlane + TM_S32 + j0, sre);
            tmem_st<32>(tlane + TM_S32 + 64 + j0, sim);
            tc_wait_st();
        }
        fence_async_smem();
        tc_fence_before();
        __syncthreads();

        SFDA_MARK(5);
        // ================= D1 = W^* S_0 and rho_1 = Qt^* S_0 (N = 128: W rows then Qt rows) ==========
        if (tid == 0) {
            tc_fence_after();
            if (ci + 1 < n_chunks) {               // staging (aliased by the solve scratch) is free again
                mbar_expect_tx(&mi.bar_in, 4 * 16384);
                tma_load_4d(smem + OFF_Q, &tm_q, &mi.bar_in, 0, h, t0 + C, b);
                tma_load_4d(smem + OFF_K, &tm_k, &mi.bar_in, 0, h, t0 + C, b);
                tma_load_4d(smem + OFF_ALPHA, &tm_alpha, &mi.bar_in, 0, h, t0 + C, b);
                tma_load_4d(smem + OFF_THETA, &tm_theta, &mi.bar_in, 0, h, t0 + C, b);
            }
            const uint32_t d_re = tmem + TM_ACC, d_im = tmem + TM_ACC + 128;
            const uint32_t s_re = tmem + TM_S16, s_im = tmem + TM_S16 + 32;
            mma_k64_ts(d_re, s_re, sbase + OFF_WQ_RE, idesc(128, 0), false);
            mma_k64_ts(d_re, s_im, sbase + OFF_WQ_IM, idesc(128, 0), true);
            mma_k64_ts(d_im, s_im, sbase + OFF_WQ_RE, idesc(128, 0), false);
            mma_k64_ts(d_im, s_re, sbase + OFF_WQ_IM, idesc(128, 1), true);
            mma_commit(&mi.bar_mma);
        }
        in_flight_in = ci + 1 < n_chunks;
        {
            const int ok_mma = mbar_wait(&mi.bar_mma, ph_mma) ? 1 : 0;
            const int ok_v = mbar_wait(&mi.bar_v, ph_v) ? 1 : 0;
            failed = __syncthreads_or((ok_mma & ok_v) ? 0 : 1);
        }
        ph_mma ^= 1;
        ph_v ^= 1;
        in_flight_v = false;
        if (failed) break;
        tc_fence_after();

        SFDA_MARK(6);
        // ================= R = V - D1 -> bf16 A operand ================================================
        {
            const int c = quad * 32 + lane;
            uint32_t r[64], pk[32];
            tmem_ld<64>(tlane + TM_ACC + 128 * half, r);
            tc_wait_ld();
            if (half == 0) {
                const __nv_bfloat16 *sv = reinterpret_cast<const __nv_bfloat16 *>(smem + OFF_V);
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    pk[i] = pack_bf16(__bfloat162float(sv[(2 * i) * DV + c]) - __uint_as_float(r[2 * i]),
                                      __bfloat162float(sv[(2 * i + 1) * DV + c]) - __uint_as_float(r[2 * i + 1]));
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) pk[i] = pack_bf16(-__uint_as_float(r[2 * i]), -__uint_as_float(r[2 * i + 1]));
            }
            tmem_st<32>(tlane + TM_X16 + 32 * half, pk);
            tc_wait_st();
        }
        tc_fence_before();
        __syncthreads();

        SFDA_MARK(7);
        // ================= E = M_beta R ================================================================
        if (tid == 0) {
            tc_fence_after();
            if (ci + 1 < n_chunks) {
                mbar_expect_tx(&mi.bar_v, 16384);
                tma_load_4d(smem + OFF_V, &tm_v, &mi.bar_v, 0, h, t0 + C, b);
            }
            const uint32_t e_re = tmem + TM_ACC, e_im = tmem + TM_ACC + 128;
            const uint32_t r_re = tmem + TM_X16, r_im = tmem + TM_X16 + 32;
            mma_k64_ts(e_re, r_re, sbase + OFF_MB_RE, idesc(64, 0), false);
            mma_k64_ts(e_re, r_im, sbase + OFF_MB_IM, idesc(64, 1), true);
            mma_k64_ts(e_im, r_im, sbase + OFF_MB_RE, idesc(64, 0), false);
            mma_k64_ts(e_im, r_re, sbase + OFF_MB_IM, idesc(64, 0), true);
            mma_commit(&mi.bar_mma);
        }
        in_flight_v = ci + 1 < n_chunks;
        failed = __syncthreads_or(mbar_wait(&mi.bar_mma, ph_mma) ? 0 : 1);
        ph_mma ^= 1;
        if (failed) break;
        tc_fence_after();
        {
            uint32_t r[64], pk[32];
            tmem_ld<64>(tlane + TM_ACC + 128 * half, r);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) pk[i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
            tmem_st<32>(tlane + TM_X16 + 32 * half, pk);
            tc_wait_st();
        }
        tc_fence_before();
        __syncthreads();

        SFDA_MARK(8);
        // ================= S += E^T Y'  and  rho += Aq E ================================================
        if (tid == 0) {
            tc_fence_after();
            const uint32_t e_re = tmem + TM_X16, e_im = tmem + TM_X16 + 32;
            const uint32_t s_re = tmem + TM_S32, s_im = tmem + TM_S32 + 64;
            mma_k64_ts(s_re, e_re, sbase + OFF_YT_RE, idesc(64, 0), true);
            mma_k64_ts(s_re, e_im, sbase + OFF_YT_IM, idesc(64, 1), true);
            mma_k64_ts(s_im, e_re, sbase + OFF_YT_IM, idesc(64, 0), true);
            mma_k64_ts(s_im, e_im, sbase + OFF_YT_RE, idesc(64, 0), true);
            const uint32_t o_re = tmem + TM_ACC + 64, o_imc = tmem + TM_ACC + 192;
            mma_k64_ts(o_re, e_re, sbase + OFF_AQ_RE, idesc(64, 0), true);
            mma_k64_ts(o_re, e_im, sbase + OFF_AQ_IM, idesc(64, 1), true);
            mma_k64_ts(o_imc, e_im, sbase + OFF_AQ_RE, idesc(64, 0), true);
            mma_k64_ts(o_imc, e_re, sbase + OFF_AQ_IM, idesc(64, 0), true);
            mma_commit(&mi.bar_mma);
        }
        failed = __syncthreads_or(mbar_wait(&mi.bar_mma, ph_mma) ? 0 : 1);
        ph_mma ^= 1;
        if (failed) break;
        tc_fence_after();

        SFDA_MARK(9);
        // ================= outputs: o = Re rho, o_im = -Im rho, staged in the (now dead) WQ tiles =======
        {
            const int c = quad * 32 + lane;
            const bool want = half ? p.o_im != nullptr : true;
            if (want) {
                uint32_t r[64];
                tmem_ld<64>(tlane + TM_ACC + 64 + 128 * half, r);
                tc_wait_ld();
                __nv_bfloat16 *stage = reinterpret_cast<__nv_bfloat16 *>(smem + (half ? OFF_WQ_IM : OFF_WQ_RE));
                const float sgn = half ? -1.f : 1.f;
#pragma unroll
                for (int t = 0; t < 64; ++t) stage[t * DV + c] = __float2bfloat16_rn(sgn * __uint_as_float(r[t]));
            }
        }
        fence_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tma_store_4d(&tm_o, smem + OFF_WQ_RE, 0, h, t0, b);
            if (p.o_im) tma_store_4d(&tm_oim, smem + OFF_WQ_IM, 0, h, t0, b);
            tma_store_commit();
        }
        SFDA_MARK(10);
    }

    if (failed) {
        if (tid == 0) atomicExch(p.status, 1u);
        // let copies that are still in flight land before the shared memory goes away
        if (in_flight_in) mbar_wait(&mi.bar_in, ph_in);
        if (in_flight_v) mbar_wait(&mi.bar_v, ph_v);
    } else if (p.S_T) {
        // final state: closing phase of the last chunk, back to paired rows
        tc_fence_after();
        const int c = quad * 32 + lane, j0 = half * 32, last = (n_chunks - 1) & 1;
        uint32_t sre[32], sim[32];
        tmem_ld<32>(tlane + TM_S32 + j0, sre);
        tmem_ld<32>(tlane + TM_S32 + 64 + j0, sim);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int j = j0 + i;
            const float cs = mi.closing_cos[last][j], sn = mi.closing_sin[last][j];
            const float xr = __uint_as_float(sre[i]), xi = __uint_as_float(sim[i]);
            p.S_T[((size_t)bh * DK + 2 * j) * DV + c] = cs * xr - sn * xi;
            p.S_T[((size_t)bh * DK + 2 * j + 1) * DV + c] = cs * xi + sn * xr;
        }
    }
    if (tid == 0) tma_store_wait_all();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem));
}

// ---- host side --------------------------------------------------------------------------------------
#ifdef SFDA_TC_TIMING
long long *g_timing = nullptr;
#endif

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = [] {
        void *f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// [B][T][H][inner] tensor, box = 64 tokens of one head.
bool make_map(CUtensorMap *map, const void *base, CUtensorMapDataType dt, int elem_bytes, int inner, int B, int T, int H)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)inner, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)inner * elem_bytes, (cuuint64_t)H * inner * elem_bytes,
                                   (cuuint64_t)T * H * inner * elem_bytes};
    const cuuint32_t box[4] = {(cuuint32_t)inner, 1, (cuuint32_t)C, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, dt, 4, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool forward_tc_supported(const ForwardArgs &a)
{
    return a.dtype == 1 && a.d_k == DK && a.d_v == DV && a.chunk == C;
}

cudaError_t launch_forward_tc(const ForwardArgs &a, uint32_t *status, cudaStream_t stream, int *launches)
{
    CUtensorMap tq, tk, tv, ta, tt, to, toi;
    if (!make_map(&tq, a.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, DK, a.B, a.T, a.H) ||
        !make_map(&tk, a.k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, DK, a.B, a.T, a.H) ||
        !make_map(&tv, a.v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, DV, a.B, a.T, a.H) ||
        !make_map(&ta, a.alpha, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, M, a.B, a.T, a.H) ||
        !make_map(&tt, a.theta, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, M, a.B, a.T, a.H) ||
        !make_map(&to, a.o, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, DV, a.B, a.T, a.H) ||
        !make_map(&toi, a.o_im ? a.o_im : a.o, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, DV, a.B, a.T, a.H))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(sfda_forward_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(status, 0, sizeof(uint32_t), stream);
    if (e != cudaSuccess) return e;
    Params p;
#ifdef SFDA_TC_TIMING
    p.timing = g_timing;
#endif
    p.beta = a.beta;
    p.S0 = a.S0;
    p.o = static_cast<__nv_bfloat16 *>(a.o);
    p.o_im = static_cast<__nv_bfloat16 *>(a.o_im);
    p.S_T = a.S_T;
    p.status = status;
    p.T = a.T;
    p.H = a.H;
    sfda_forward_tc_kernel<<<(unsigned)(a.B * a.H), kThreads, kSmemBytes, stream>>>(tq, tk, tv, ta, tt, to, toi, p);
    e = cudaGetLastError();
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace sfda
