// sfda_chunk_factors: per-chunk factors of P = A_C ... A_1 = Gamma - Y M W^* (Theorem "Constructive left-to-right
// chunk-WY recursion", Cor. "SFDA admits exact constructive block-WY products") in fp32 on the CUDA cores.
//
// With gamma_t = prod_{s<=t} lambda_s = a_t e^{i phi_t} inside the chunk and k'_t = e^{-i phi_t} k_t:
//
//   Gamma = gamma_C,   W[:,t] = conj(gamma_t) k_t = a_t k'_t,   Y[:,t] = (gamma_C / gamma_t) beta_t k_t
//   N[t][i] = beta_i k_t^* diag(gamma_t / gamma_i) k_i = beta_i sum_j conj(k'_tj) k'_ij a_tj / a_ij   (i < t)
//   M = (I + N)^{-1}                                                       (Eq. "constructive-M" unrolled)
//
// One CTA of 256 threads per chunk, three CTAs per SM; everything after the loads lives in shared memory (N and its
// inverse take the place of the rotated keys once the Gram sums are in registers):
//   A  scan:     thread = (coordinate j, group of C/G tokens): log-decay and integer-phase prefix sums, rotated keys
//   B  export:   Gamma, W, Y (coalesced over t)
//   C  Gram:     pairs (t, i) of different 8-token blocks on the tensor cores (mma.sync, 3 x TF32), level by level
//                of a binary split of the chunk, the decay split at the last token r of the lower half:
//                a_t/a_i = (a_t/a_r)(a_r/a_i), both factors <= 1, so nothing overflows whatever alpha is; pairs
//                inside a block take the ratio directly: one warp per block, the block's tokens in registers,
//                packed two-lane arithmetic, sums over the lanes through a small scratch.
//   D  inverse:  8 x 8 diagonal blocks by substitution, then X = [[X11, 0], [-X22 N21 X11, X22]] doubling the
//                block size until it is C, both products of a level as 16 x 8 tiles on the tensor cores (3 x TF32).
// Only ratios <= 1 are ever formed, so any alpha in [0, 1] is safe.  Offsets inside a chunk are 32-bit: with 64-bit
// offsets the unrolled loads and stores of the scan spent more instructions on addresses than on data.
#include "sfda_common.cuh"
#include "sfda_internal.h"

namespace sfda {
namespace {

constexpr int kFacThreads = 256;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// log2 of a decay factor, floored like log_decay (e^-30 = 2^-43.28): one special-function instruction, absolute
// error about 2^-22.
__device__ __forceinline__ float log2_decay(float alpha)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(alpha));
    return fmaxf(y, -30.0f * kLog2e);
}

// Two adjacent elements (real and imaginary part of one coordinate) in one load.
__device__ __forceinline__ float2 ld_pair(const float *p, size_t i) { return *reinterpret_cast<const float2 *>(p + i); }
__device__ __forceinline__ float2 ld_pair(const __nv_bfloat16 *p, size_t i)
{
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(p + i));
}

// cos / sin of a phase given in 2^-32 turns: the top 23 bits as a fraction of a turn in [-1/2, 1/2), fast sine.
__device__ __forceinline__ void turns_cos_sin_fast(uint32_t turns, float *c, float *s)
{
    float f = __uint_as_float(0x3f800000u | (turns >> 9)) - 1.0f;
    f -= f >= 0.5f ? 1.0f : 0.0f;
    __sincosf(f * 6.283185307f, s, c);
}

// x = head + tail to within 2^-20 |x|: the head is x cut to TF32's ten mantissa bits, the tail the exact rest, of which
// the tensor core in turn reads the leading bits (it ignores the low 13 bits of a TF32 operand).  Two instructions.
__device__ __forceinline__ void split_tf32(float x, uint32_t &head, uint32_t &tail)
{
    head = __float_as_uint(x) & 0xffffe000u;
    tail = __float_as_uint(x - __uint_as_float(head));
}
__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2])
{
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
// d += a b^T with fp32-like accuracy: the small products first
__device__ __forceinline__ void mma3_tf32(float (&d)[4], const uint32_t (&ah)[4], const uint32_t (&al)[4],
                                          const uint32_t (&bh)[2], const uint32_t (&bl)[2])
{
    mma_tf32(d, al, bh);
    mma_tf32(d, ah, bl);
    mma_tf32(d, ah, bh);
}
template <int DK, int C>
struct FacSmem {
    static constexpr int M = DK / 2;
    static constexpr int KS = M + 1;        // row stride of kp in float2 (odd: rows and columns both conflict-free)
    static constexpr int LS = M + 1;        // row stride of lg2 in floats
    static constexpr int NS = C + 4;        // row stride of N / X in float2 (4 mod 16: the tensor-core tiles' 64-bit loads
                                            // of a half-warp, rows g and columns c or rows c and columns g, hit 16 different slots)
    static constexpr int G = kFacThreads / M;   // token groups of the scan
    static constexpr int TG = C / G;            // tokens per group
    static constexpr int kKeyRows = C * (KS > NS ? KS : NS);   // float2: the larger of k' and N
    static constexpr int kGrpFloats = 2 * G * M > 2 * (C / 8) * 28 ? 2 * G * M : 2 * (C / 8) * 28;
    static constexpr size_t bytes = (size_t)kKeyRows * 8 + (size_t)C * LS * 4 + (size_t)kGrpFloats * 4 +
                                    (size_t)M * 12 + (size_t)C * 4 + (size_t)(kFacThreads / 32) * 14 * 33 * 4;
    float2 *kp;        // [C][KS] rotated keys k' until the Gram sums are in registers ...
    float2 *nx;        // ... then [C][NS] N, inverted in place (same memory)
    float *lg2;        // [C][LS] log2 of a_t; after the Gram: scratch of the inverse's products
    float *grp_lg;     // [G][M] group totals of the scan; later the Gram sums of the pairs inside 8-token blocks
    uint32_t *grp_tu;  // [G][M]
    float *gcr, *gci, *lg2C;   // [M] e^{i phi_C}, log2 a_C
    float *beta;       // [C]
    float *red;        // [warp][14][33] terms of seven pairs inside a block, lane by lane
    __device__ explicit FacSmem(unsigned char *base)
    {
        kp = reinterpret_cast<float2 *>(base);
        nx = kp;
        lg2 = reinterpret_cast<float *>(kp + kKeyRows);
        grp_lg = lg2 + C * LS;
        grp_tu = reinterpret_cast<uint32_t *>(grp_lg + G * M);
        gcr = grp_lg + kGrpFloats;
        gci = gcr + M;
        lg2C = gci + M;
        beta = lg2C + M;
        red = beta + C;
    }
};
static_assert(FacSmem<128, 64>::bytes <= 74 * 1024, "three CTAs per SM need at most 75 KB each");

// One 8-wide step of a complex 16 x 8 tile product on the tensor cores with fp32-like accuracy (3 x TF32 per real
// product).  `a` points at element (row g, column c) of the A tile's columns of this step, `b` at element
// (row c, column g) of the B tile's rows (g = lane / 4, c = lane % 4); strides in float2.  The four real products
// keep their own accumulators: Re = acc[0] - acc[1], Im = acc[2] + acc[3].
__device__ __forceinline__ void cmma3_step(float (&acc)[4][4], const float2 *a, int as, const float2 *b, int bs)
{
    uint32_t arh[4], arl[4], aih[4], ail[4], brh[2], brl[2], bih[2], bil[2];
#pragma unroll
    for (int e = 0; e < 4; ++e) {          // a0 (g, c), a1 (g + 8, c), a2 (g, c + 4), a3 (g + 8, c + 4)
        const float2 v = a[(e & 1) * 8 * as + (e >> 1) * 4];
        split_tf32(v.x, arh[e], arl[e]);
        split_tf32(v.y, aih[e], ail[e]);
    }
#pragma unroll
    for (int e = 0; e < 2; ++e) {          // b0 (k = c, n = g), b1 (k = c + 4, n = g)
        const float2 v = b[e * 4 * bs];
        split_tf32(v.x, brh[e], brl[e]);
        split_tf32(v.y, bih[e], bil[e]);
    }
    mma3_tf32(acc[0], arh, arl, brh, brl);
    mma3_tf32(acc[1], aih, ail, bih, bil);
    mma3_tf32(acc[2], arh, arl, bih, bil);
    mma3_tf32(acc[3], aih, ail, brh, brl);
}

// One level of the block inverse: every pair of finished diagonal blocks of size HS (X11 at o, X22 at o + HS, N21
// below X11) becomes one of size 2 HS: X21 = -X22 (N21 X11), both products as 16 x 8 tiles on the tensor cores, one
// tile per warp and round.  Whole 8 x 8 blocks are read: the blocks on the diagonal hold zeros above it, the block
// right of the upper diagonal block of every 16 rows was zeroed, and the ranges of the sums leave out every other
// block above the diagonal.  With HS = 8 the tile lies on the whole 16-row block and its lower eight rows count.
template <typename S, int C, int HS>
__device__ __forceinline__ void merge_level(const S &sm, int tid)
{
    if constexpr (HS < C) {
        constexpr int PS = 36;                              // row stride of the scratch (float2): conflict-free 64-bit loads
        constexpr int MT = HS >= 16 ? HS / 16 : 1, NT = HS / 8, kTiles = (C / (2 * HS)) * MT * NT;
        static_assert((C / 2) * PS * 8 <= (C * S::LS + S::kGrpFloats) * 4, "the products' scratch must fit where lg2 and the group sums were");
        float2 *P = reinterpret_cast<float2 *>(sm.lg2);    // [merge][HS][PS]: N21 X11 (the decays and the group sums after them are done)
        const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
        for (int tile = warp; tile < kTiles; tile += kFacThreads / 32) {
            const int mg = tile / (MT * NT), mt = (tile % (MT * NT)) / NT, nt = tile % NT, o = mg * 2 * HS;
            const int arow = HS >= 16 ? o + HS + 16 * mt : o;
            float acc[4][4];
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
            const float2 *a = sm.nx + (arow + g) * S::NS + o + c;
            const float2 *b = sm.nx + (o + c) * S::NS + o + 8 * nt + g;
#pragma unroll 1
            for (int ks = nt; ks < NT; ++ks)                // X11[k][col] = 0 for k-blocks above the column's
                cmma3_step(acc, a + 8 * ks, S::NS, b + 8 * ks * S::NS, S::NS);
            float2 *dst = P + (mg * HS + 16 * mt + g) * PS + 8 * nt + 2 * c;
            if (HS >= 16)
                *reinterpret_cast<float4 *>(dst) = make_float4(acc[0][0] - acc[1][0], acc[2][0] + acc[3][0],
                                                               acc[0][1] - acc[1][1], acc[2][1] + acc[3][1]);
            *reinterpret_cast<float4 *>(dst + (HS >= 16 ? 8 * PS : 0)) =
                make_float4(acc[0][2] - acc[1][2], acc[2][2] + acc[3][2], acc[0][3] - acc[1][3], acc[2][3] + acc[3][3]);
        }
        __syncthreads();
        for (int tile = warp; tile < kTiles; tile += kFacThreads / 32) {
            const int mg = tile / (MT * NT), mt = (tile % (MT * NT)) / NT, nt = tile % NT, o = mg * 2 * HS;
            const int arow = HS >= 16 ? o + HS + 16 * mt : o;
            float acc[4][4];
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
            const float2 *a = sm.nx + (arow + g) * S::NS + o + HS + c;
            const float2 *b = P + (mg * HS + c) * PS + 8 * nt + g;
            const int nks = HS >= 16 ? 2 * mt + 2 : 1;      // X22[row][k] = 0 for k-blocks beyond the tile's rows
#pragma unroll 1
            for (int ks = 0; ks < nks; ++ks) cmma3_step(acc, a + 8 * ks, S::NS, b + 8 * ks * PS, PS);
            float2 *dst = sm.nx + (o + HS + 16 * mt + g) * S::NS + o + 8 * nt + 2 * c;
            if (HS >= 16)
                *reinterpret_cast<float4 *>(dst) = make_float4(acc[1][0] - acc[0][0], -acc[2][0] - acc[3][0],
                                                               acc[1][1] - acc[0][1], -acc[2][1] - acc[3][1]);
            *reinterpret_cast<float4 *>(dst + (HS >= 16 ? 8 * S::NS : 0)) =
                make_float4(acc[1][2] - acc[0][2], -acc[2][2] - acc[3][2], acc[1][3] - acc[0][3], -acc[2][3] - acc[3][3]);
        }
        __syncthreads();
    }
}

template <int DK, int C, typename T>
__global__ void __launch_bounds__(kFacThreads, 3)
sfda_chunk_factors_kernel(const T *__restrict__ k, const float *__restrict__ alpha, const float *__restrict__ theta,
                          const float *__restrict__ beta, float *__restrict__ Gamma, float *__restrict__ Y,
                          float *__restrict__ Mo, float *__restrict__ W, uint32_t *__restrict__ turns_out, int T_,
                          int H, int NC, int sup)
{
    using S = FacSmem<DK, C>;
    constexpr int M = S::M, G = S::G, TG = S::TG;
    static_assert(C % 8 == 0 && C % G == 0 && TG >= 1, "chunk must split into the scan's groups and 8-token blocks");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const S sm(smem_raw);

    const int tid = threadIdx.x;
    const int ci = blockIdx.x % NC;
    const int bh = blockIdx.x / NC;
    const int h = bh % H, b = bh / H;
    const int t0 = ci * C;
    const int len = min(C, T_ - t0);
    // The factors of chunk `ci` go to tile `part` of output chunk `sc`, which spans `sup` tiles (sup = 1: the chunk is
    // the tile; sup = 2: a 128-token chunk out of two tiles, completed by sfda_compose_factors_kernel).
    const int sc = ci / sup, part = ci - sc * sup, Co = sup * C;
    const size_t out_id = (size_t)bh * ((NC + sup - 1) / sup) + sc;

    // ---- A: loads and scan.  Tokens past `len` are neutral (alpha = 1, theta = 0, beta = 0, k = 0).
    {
        const int j = tid % M, g = tid / M;
        float lgv[TG];
        uint32_t tu[TG];
        float2 kv[TG];
        const size_t row0 = ((size_t)b * T_ + t0 + g * TG) * H + h;      // first token of the group
        const float *ap = alpha + row0 * M + j, *tp = theta + row0 * M + j;
        const T *kq = k + row0 * DK + 2 * j;
        // coordinates from one token to the next; offsets inside a chunk stay below 2^32, and 32-bit offsets keep
        // the address arithmetic of the unrolled loads to one instruction each
        const unsigned cs = (unsigned)H * M;
        uint32_t *tpo = turns_out ? turns_out + row0 * M + j : nullptr;
#pragma unroll
        for (int x = 0; x < TG; ++x) {
            const int t = g * TG + x;
            float al = 1.f, th = 0.f;
            kv[x] = make_float2(0.f, 0.f);
            if (t < len) {
                al = ap[x * cs];
                th = tp[x * cs];
                kv[x] = ld_pair(kq, (size_t)(2u * x * cs));
            }
            lgv[x] = al;
            tu[x] = __float_as_uint(th);
        }
        if (tid < C) sm.beta[tid] = tid < len ? beta[((size_t)b * T_ + t0 + tid) * H + h] : 0.f;
        float acc = 0.f;
        uint32_t ta = 0u;
#pragma unroll
        for (int x = 0; x < TG; ++x) {     // inclusive prefixes inside the group
            acc += log2_decay(lgv[x]);
            ta += phase_to_turns(__uint_as_float(tu[x]));
            lgv[x] = acc;
            tu[x] = ta;
        }
        sm.grp_lg[g * M + j] = acc;
        sm.grp_tu[g * M + j] = ta;
        __syncthreads();
        float base = 0.f;
        uint32_t tb = 0u;
        for (int gg = 0; gg < g; ++gg) {
            base += sm.grp_lg[gg * M + j];
            tb += sm.grp_tu[gg * M + j];
        }
#pragma unroll
        for (int x = 0; x < TG; ++x) {
            const int t = g * TG + x;
            const float l = base + lgv[x];
            const uint32_t tt = tb + tu[x];
            if (tpo && t < len) tpo[x * cs] = tt;
            float cs, sn;
            turns_cos_sin_fast(tt, &cs, &sn);
            sm.lg2[t * S::LS + j] = l;
            sm.kp[t * S::KS + j] = make_float2(kv[x].x * cs + kv[x].y * sn, kv[x].y * cs - kv[x].x * sn);   // e^{-i phi} k
            if (t == C - 1) {
                turns_to_cos_sin(tt, &cs, &sn);    // the exported Gamma takes the accurate sine
                sm.gcr[j] = cs;
                sm.gci[j] = sn;
                sm.lg2C[j] = l;
            }
        }
    }
    __syncthreads();

    // ---- B: Gamma, W, Y
    if (Gamma) {
        for (int j = tid; j < M; j += kFacThreads) {
            const float a = ex2f(sm.lg2C[j]);
            const float2 gam = make_float2(a * sm.gcr[j], a * sm.gci[j]);
            if (sup == 1) reinterpret_cast<float2 *>(Gamma)[out_id * M + j] = gam;
            // a tile's Gamma waits in a block of M above the diagonal, which ends up zero: tile 0 in row 1 of block
            // (0, 1), tile b >= 1 in row 0 of block (0, b)
            else reinterpret_cast<float2 *>(Mo)[(part == 0 ? out_id * Co + 1 : out_id * Co) * Co + (part == 0 ? C : part * C) + j] = gam;
        }
    }
    if (W || Y) {
        // a thread keeps its token and walks over the coordinates: consecutive lanes store consecutive tokens
        constexpr int JS = kFacThreads / C;                 // coordinates per sweep of the CTA
        const int t = tid % C;
        const float bt = sm.beta[t];
        float2 *Wp = reinterpret_cast<float2 *>(W) + (out_id * M + tid / C) * Co + part * C + t;
        float2 *Yp = reinterpret_cast<float2 *>(Y) + (out_id * M + tid / C) * Co + part * C + t;
#pragma unroll 4
        for (int j = tid / C; j < M; j += JS, Wp += JS * Co, Yp += JS * Co) {
            const float2 kk = sm.kp[t * S::KS + j];
            const float l = sm.lg2[t * S::LS + j];
            if (W) {   // W[:,t] = conj(gamma_t) k_t = a_t k'_t
                const float a = ex2f(l);
                *Wp = make_float2(a * kk.x, a * kk.y);
            }
            if (Y) {   // Y[:,t] = (gamma_C / gamma_t) beta_t k_t = (a_C / a_t) e^{i phi_C} beta_t k'_t
                const float w = bt * ex2f(sm.lg2C[j] - l);
                const float gr = sm.gcr[j], gi = sm.gci[j];
                *Yp = make_float2(w * (gr * kk.x - gi * kk.y), w * (gr * kk.y + gi * kk.x));
            }
        }
    }

    // ---- C: N[t][i] = beta_i sum_j conj(k'_tj) k'_ij a_tj / a_ij,  i < t
    if (Mo) {
        constexpr int NB = C / 8;                          // blocks of 8 tokens
        constexpr int kPairs = NB * 28;                    // pairs (t, i), i < t, inside the blocks
        // Pairs of different blocks, on the tensor cores (mma.sync m16n8k8, 3 x TF32: every operand is split into
        // a TF32 head and a TF32 tail and the three significant products are added in fp32, which keeps the sums
        // at fp32 accuracy).  The pairs are taken level by level of a binary split of the chunk: rows of the upper
        // half of a span of 16, 32 or 64 tokens against the columns of its lower half, with the decay split at the
        // last token r of the lower half, a_t / a_i = (a_t / a_r)(a_r / a_i), both factors <= 1.  Job = a tile of
        // 16 rows x 8 columns with its r; rows of the tile that do not lie past r are computed (decay clamped to
        // 1) and dropped.  A warp has at most two jobs, which share their row operand when tile and r agree.
        // The sums stay in registers: N will overwrite the keys once everybody has read them.
        const int warp = tid >> 5, lane = tid & 31, fg = lane >> 2, ft = lane & 3;
        // Pairs inside a block take the decay ratio directly: a_t / a_i <= 1 for i < t.  One warp per block; a lane keeps
        // the eight tokens' rotated keys and log-decays of its coordinates (lane and lane + 32) in registers and forms
        // the 28 pairs' terms with packed two-lane arithmetic; the sums over the lanes go through a small scratch,
        // seven pairs at a time.  The results wait in the scan's group totals, which are no longer needed.
        float2 *dg = reinterpret_cast<float2 *>(sm.grp_lg);
        for (int blk = warp; blk < NB; blk += kFacThreads / 32) {
            float2 kx[8], ky[8], lg[8];                    // .x: coordinate `lane`, .y: coordinate `lane + 32`
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const float2 k0 = sm.kp[(8 * blk + r) * S::KS + lane];
                float2 k1 = make_float2(0.f, 0.f);
                float l1 = 0.f;
                if (M > 32) {
                    k1 = sm.kp[(8 * blk + r) * S::KS + (M > 32 ? lane + 32 : lane)];
                    l1 = sm.lg2[(8 * blk + r) * S::LS + (M > 32 ? lane + 32 : lane)];
                }
                kx[r] = make_float2(k0.x, k1.x);
                ky[r] = make_float2(k0.y, k1.y);
                lg[r] = make_float2(sm.lg2[(8 * blk + r) * S::LS + lane], l1);
            }
            float *red = sm.red + warp * (14 * 33);
#pragma unroll
            for (int t = 1; t < 8; ++t) {
                const float2 nky = make_float2(-ky[t].x, -ky[t].y);
#pragma unroll
                for (int i = 0; i < t; ++i) {
                    const int pidx = t * (t - 1) / 2 + i, v = 2 * (pidx % 7);   // compile-time
                    const float2 d = __fadd2_rn(lg[t], make_float2(-lg[i].x, -lg[i].y));
                    const float2 w = make_float2(ex2f(d.x), ex2f(d.y));
                    const float2 pr = __ffma2_rn(ky[t], ky[i], __fmul2_rn(kx[t], kx[i]));      // Re conj(k'_t) k'_i
                    const float2 pi = __ffma2_rn(nky, kx[i], __fmul2_rn(kx[t], ky[i]));        // Im conj(k'_t) k'_i
                    const float2 sr = __fmul2_rn(w, pr), si = __fmul2_rn(w, pi);
                    red[v * 33 + lane] = sr.x + sr.y;
                    red[(v + 1) * 33 + lane] = si.x + si.y;
                    if (pidx % 7 == 6) {                   // seven pairs are in: add up over the lanes
                        __syncwarp();
                        // lanes 2 v and 2 v + 1 add the two halves of value v's 32 terms
                        float acc = 0.f;
                        const float *src = red + (lane >> 1) * 33 + 16 * (lane & 1);
                        if (lane < 28) {
#pragma unroll
                            for (int x = 0; x < 16; ++x) acc += src[x];
                        }
                        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
                        const float im = __shfl_xor_sync(0xffffffffu, acc, 2);
                        if ((lane & 3) == 0 && lane < 28) dg[(pidx - 6 + (lane >> 2)) * NB + blk] = make_float2(acc, im);
                        __syncwarp();
                    }
                }
            }
        }
        int jm[2] = {-1, -1}, jc[2] = {0, 0}, jr[2] = {0, 0};   // row tile, first column, split token of the jobs
        if (C == 64) {
            if (warp < 4) { jm[0] = jm[1] = 2 + (warp >> 1); jc[0] = 16 * (warp & 1); jc[1] = jc[0] + 8; jr[0] = jr[1] = 31; }
            else if (warp < 6) { jm[0] = jm[1] = 2 * warp - 7; jc[0] = 32 * (warp - 4); jc[1] = jc[0] + 8; jr[0] = jr[1] = jc[0] + 15; }
            else { jm[0] = 2 * (warp - 6); jm[1] = jm[0] + 1; jc[0] = 16 * jm[0]; jc[1] = 16 * jm[1]; jr[0] = jc[0] + 7; jr[1] = jc[1] + 7; }
        } else if (C == 32) {
            if (warp == 0) { jm[0] = jm[1] = 1; jc[0] = 0; jc[1] = 8; jr[0] = jr[1] = 15; }
            else if (warp < 3) { jm[0] = warp - 1; jc[0] = 16 * jm[0]; jr[0] = jc[0] + 7; }
        } else {
            if (warp == 0) { jm[0] = 0; jc[0] = 0; jr[0] = 7; }
        }
        const bool share = jm[1] == jm[0] && jr[1] == jr[0];
        float acc[2][3][4];                                // per job: Re, and the two parts of Im = sum ar bi - sum ai br
#pragma unroll
        for (int n = 0; n < 2; ++n)
#pragma unroll
            for (int x = 0; x < 3; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[n][x][y] = 0.f;
        if (jm[0] >= 0) {
#pragma unroll 1
            for (int ks = 0; ks < M / 8; ++ks) {
                // the 8 coordinates of this step, chosen so that the 64-bit loads of a half-warp hit 16 different
                // banks: fragment column c <-> coordinate jb + 4 (c % 4) + c / 4
                const int jb = 16 * (ks >> 1) + 2 * (ks & 1) + 4 * ft;
                uint32_t ah[2][4], al[2][4], bh_[2][2], bl[2][2];   // [re / im][fragment element], heads and tails
#pragma unroll
                for (int n = 0; n < 2; ++n) {
                    if (n == 1 && jm[1] < 0) break;
                    const int r = jr[n];
                    if (n == 0 || !share) {
                        const int rowA = 16 * jm[n] + fg;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {      // a0 (g, c), a1 (g + 8, c), a2 (g, c + 4), a3 (g + 8, c + 4)
                            const int row = rowA + 8 * (e & 1), j = jb + (e >> 1);
                            const float w = ex2f(fminf(sm.lg2[row * S::LS + j] - sm.lg2[r * S::LS + j], 0.f));
                            const float2 kk = sm.kp[row * S::KS + j];
                            split_tf32(w * kk.x, ah[0][e], al[0][e]);
                            split_tf32(w * kk.y, ah[1][e], al[1][e]);
                        }
                    }
                    const int rowB = jc[n] + fg;
#pragma unroll
                    for (int e = 0; e < 2; ++e) {          // b0 (k = c, n = g), b1 (k = c + 4, n = g)
                        const int j = jb + e;
                        const float w = ex2f(sm.lg2[r * S::LS + j] - sm.lg2[rowB * S::LS + j]);   // a_r / a_i <= 1
                        const float2 kk = sm.kp[rowB * S::KS + j];
                        split_tf32(w * kk.x, bh_[0][e], bl[0][e]);
                        split_tf32(w * kk.y, bh_[1][e], bl[1][e]);
                    }
                    mma3_tf32(acc[n][0], ah[0], al[0], bh_[0], bl[0]);   // ar br
                    mma3_tf32(acc[n][0], ah[1], al[1], bh_[1], bl[1]);   // ai bi
                    mma3_tf32(acc[n][1], ah[0], al[0], bh_[1], bl[1]);   // ar bi
                    mma3_tf32(acc[n][2], ah[1], al[1], bh_[0], bl[0]);   // ai br
                }
            }
        }
        __syncthreads();           // every read of the keys is done: N goes where they were
        // the 8 x 8 block right of the upper diagonal block of every 16 rows: read as zeros by the inverse's tiles
        for (int idx = tid; idx < (C / 16) * 64; idx += kFacThreads)
            sm.nx[(16 * (idx >> 6) + ((idx >> 3) & 7)) * S::NS + 16 * (idx >> 6) + 8 + (idx & 7)] = make_float2(0.f, 0.f);
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            if (jm[n] < 0) continue;
#pragma unroll
            for (int e = 0; e < 4; ++e) {                  // c0 (g, 2c), c1 (g, 2c + 1), c2 (g + 8, 2c), c3 (g + 8, 2c + 1)
                const int row = 16 * jm[n] + fg + 8 * (e >> 1), i = jc[n] + 2 * ft + (e & 1);
                if (row > jr[n]) {
                    const float bt = sm.beta[i];
                    sm.nx[row * S::NS + i] = make_float2(bt * acc[n][0][e], bt * (acc[n][1][e] - acc[n][2][e]));
                }
            }
        }
        for (int pr_ = tid; pr_ < kPairs; pr_ += kFacThreads) {
            const int blk = pr_ % NB, pidx = pr_ / NB;
            int t = 1;
            while (t * (t + 1) / 2 <= pidx) ++t;
            const int i = pidx - t * (t - 1) / 2;
            const float2 v = dg[pr_];
            const float bt = sm.beta[8 * blk + i];
            sm.nx[(8 * blk + t) * S::NS + 8 * blk + i] = make_float2(bt * v.x, bt * v.y);
        }
        __syncthreads();

        // ---- D: X = (I + N)^{-1} in place.  Diagonal 8 x 8 blocks: thread = (block, column c), right-looking
        // substitution of (I + N) x = e_c in registers; everybody reads before anybody writes.
        {
            float xr[8], xi[8];
            const int blk = tid >> 3, c = tid & 7, o = 8 * blk;
            if (tid < C) {
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    xr[r] = r == c ? 1.f : 0.f;
                    xi[r] = 0.f;
                }
#pragma unroll
                for (int i = 0; i < 7; ++i) {
                    const float vr = xr[i], vi = xi[i];
#pragma unroll
                    for (int r = i + 1; r < 8; ++r) {
                        const float2 n = sm.nx[(o + r) * S::NS + o + i];
                        xr[r] -= n.x * vr - n.y * vi;
                        xi[r] -= n.x * vi + n.y * vr;
                    }
                }
            }
            __syncthreads();
            if (tid < C) {
#pragma unroll
                for (int r = 0; r < 8; ++r) sm.nx[(o + r) * S::NS + o + c] = make_float2(xr[r], xi[r]);
            }
            __syncthreads();
        }
        // merges: blocks of size HS at o (X11) and o + HS (X22), N21 below X11:  X21 = -X22 (N21 X11)
        merge_level<S, C, 8>(sm, tid);
        merge_level<S, C, 16>(sm, tid);
        merge_level<S, C, 32>(sm, tid);
        for (int idx = tid; idx < C * C; idx += kFacThreads) {
            const int t = idx / C, i = idx % C;
            reinterpret_cast<float2 *>(Mo)[(out_id * Co + part * C + t) * Co + part * C + i] =
                i <= t ? sm.nx[t * S::NS + i] : make_float2(0.f, 0.f);
        }
    }
}

template <int DK, int C, typename T>
cudaError_t launch_fac(const FactorArgs &a, cudaStream_t stream, int sup = 1)
{
    constexpr size_t smem = FacSmem<DK, C>::bytes;
    auto kern = sfda_chunk_factors_kernel<DK, C, T>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int NC = (a.T + C - 1) / C;
    const unsigned grid = (unsigned)a.B * a.H * NC;
    kern<<<grid, kFacThreads, smem, stream>>>(static_cast<const T *>(a.k), a.alpha, a.theta, a.beta, a.Gamma, a.Y, a.M,
                                              a.W, a.phase_turns, a.T, a.H, NC, sup);
    return cudaGetLastError();
}

// Factors of a chunk of 128 or 256 tokens out of those of its 64-token tiles (Section 6, "superchunks"; the block
// form of Eq. "constructive-M").  Appending a tile b with P_b = Gamma_b - Y_b M_b W_b^* to a prefix of tiles with
// P_p = Gamma_p - Y_p M_p W_p^* gives
//
//   P_b P_p = Gamma - Y M W^*,   Gamma = Gamma_b Gamma_p,   Y = [Gamma_b Y_p | Y_b],   W = [W_p | Gamma_p^* W_b],
//   M = [[M_p, 0], [-M_b (W_b^* Y_p) M_p, M_b]],
//
// exact, and every factor is a product of numbers of modulus at most one.  The tile kernel has left every tile's Y,
// W and M at their places in the chunk's layout and the tiles' Gamma in the blocks of M above the diagonal (tile 0:
// row 1 of block (0, 1); tile b >= 1: row 0 of block (0, b)).  This kernel, launched once per appended tile
// b = 1 .. sup - 1 with one CTA per chunk, forms block row b of M left of the diagonal,
// X_c = -M_b sum_{k >= c} Z_k M_p[k][c] with Z_k = W_b^* Y_p[:, block k], as 16 x 8 tiles on the tensor cores
// (3 x TF32) through shared memory, scales the prefix's Y by Gamma_b and W_b by conj(Gamma_p), zeroes the blocks above
// tile b's diagonal block, keeps the running Gamma in the output array and adds the prefix's closing phase to the
// integer phases of tile b's tokens.  A tile without tokens (the sequence ends before it) becomes the neutral tile:
// zero columns, identity block.
constexpr int kCmpThreads = 512;
constexpr int kCmpStride = 68;                              // float2 row stride of the 64 x 64 regions (4 mod 16)
constexpr size_t compose_smem_bytes(int DK, int b) { return (size_t)(b + 2) * 64 * kCmpStride * 8 + (size_t)DK * 8; }
template <int DK>
__global__ void __launch_bounds__(kCmpThreads)
sfda_compose_factors_kernel(float *__restrict__ Gamma, float *__restrict__ Y, float *__restrict__ Mo,
                            float *__restrict__ W, uint32_t *__restrict__ turns, int T_, int H, int NCo, int sup, int b)
{
    constexpr int M = DK / 2, h = 64, RS = kCmpStride;
    const int Co = h * sup, P = h * b;                     // chunk length, prefix length
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float2 *ra = reinterpret_cast<float2 *>(smem_raw), *rb = ra + 64 * RS, *zs = rb + 64 * RS;   // zs: b regions
    float2 *gb = zs + b * 64 * RS, *gp = gb + M;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
    const size_t out_id = blockIdx.x;
    const int bh = (int)(out_id / NCo), sc = (int)(out_id % NCo), bb = bh / H, hh = bh % H;
    const int t0 = sc * Co;
    const bool has = t0 + P < T_;                          // tile b holds at least one token
    float2 *Y2 = reinterpret_cast<float2 *>(Y) + out_id * M * Co, *W2 = reinterpret_cast<float2 *>(W) + out_id * M * Co;
    float2 *M2 = reinterpret_cast<float2 *>(Mo) + out_id * Co * Co, *G2 = reinterpret_cast<float2 *>(Gamma) + out_id * M;
    auto cmul = [](float2 x, float2 y) { return make_float2(x.x * y.x - x.y * y.y, x.x * y.y + x.y * y.x); };
    // one 64 x 64 complex product as 32 tiles of 16 x 8 (two per warp), 3 x TF32, k-steps ks0(tile) .. ks1(tile) - 1;
    // `put` receives every result element
    auto product = [&](const float2 *A, const float2 *Bm, auto ks0, auto ks1, auto put) {
        for (int tile = warp; tile < 32; tile += kCmpThreads / 32) {
            const int mt = tile >> 3, nt = tile & 7;
            float acc[4][4];
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
            const int k1 = ks1(mt, nt);
#pragma unroll 1
            for (int ks = ks0(mt, nt); ks < k1; ++ks)
                cmma3_step(acc, A + (16 * mt + g) * RS + 8 * ks + c, RS, Bm + (8 * ks + c) * RS + 8 * nt + g, RS);
#pragma unroll
            for (int e = 0; e < 4; ++e)        // c0 (g, 2c), c1 (g, 2c + 1), c2 (g + 8, 2c), c3 (g + 8, 2c + 1)
                put(16 * mt + g + 8 * (e >> 1), 8 * nt + 2 * c + (e & 1), make_float2(acc[0][e] - acc[1][e], acc[2][e] + acc[3][e]));
        }
    };
    auto load_block = [&](float2 *dst, int row0, int col0) {   // a 64 x 64 block of M
        for (int i = tid; i < h * h; i += kCmpThreads) dst[(i / h) * RS + i % h] = M2[(size_t)(row0 + i / h) * Co + col0 + i % h];
    };

    for (int j = tid; j < M; j += kCmpThreads) {
        gb[j] = has ? M2[P + j] : make_float2(1.f, 0.f);                 // tile b: row 0 of block (0, b)
        gp[j] = b == 1 ? M2[Co + h + j] : G2[j];                         // tile 0: row 1 of block (0, 1); else the running one
    }
    if (has) {
        for (int i = tid; i < M * h; i += kCmpThreads) {     // W_b^* -> rb[t][j]
            const int j = i / h, t = i % h;
            const float2 w = W2[j * Co + P + t];
            rb[t * RS + j] = make_float2(w.x, -w.y);
        }
#pragma unroll 1
        for (int cb = 0; cb < b; ++cb) {                     // Z_cb = W_b^* Y_p[:, block cb]  (sum over the m coordinates)
            __syncthreads();                                 // (the previous block's products have read ra)
            for (int i = tid; i < M * h; i += kCmpThreads) ra[(i / h) * RS + i % h] = Y2[(i / h) * Co + h * cb + i % h];
            __syncthreads();
            float2 *z = zs + cb * 64 * RS;
            product(rb, ra, [](int, int) { return 0; }, [](int, int) { return M / 8; },
                    [&](int r, int cc, float2 v) { z[r * RS + cc] = v; });
            for (int i = tid; i < M * h; i += kCmpThreads)   // Y_p <- Gamma_b Y_p (from the copy in shared memory)
                Y2[(i / h) * Co + h * cb + i % h] = cmul(gb[i / h], ra[(i / h) * RS + i % h]);
        }
        for (int i = tid; i < M * h; i += kCmpThreads) {     // W_b <- conj(Gamma_p) W_b = conj(Gamma_p conj(W_b))
            const int j = i / h, t = i % h;
            const float2 w = cmul(gp[j], rb[t * RS + j]);
            W2[j * Co + P + t] = make_float2(w.x, -w.y);
        }
#pragma unroll 1
        for (int cb = 0; cb < b; ++cb) {
            // T = sum_{k >= cb} Z_k M_p[k][cb] into rb (the diagonal block of M_p is lower triangular: k-steps from the
            // column's on), then X_cb = -M_b T (M_b is lower triangular: k-steps up to the rows')
#pragma unroll 1
            for (int k = cb; k < b; ++k) {
                __syncthreads();
                load_block(ra, h * k, h * cb);
                __syncthreads();
                const float2 *z = zs + k * 64 * RS;
                if (k == cb)
                    product(z, ra, [](int, int nt) { return nt; }, [](int, int) { return 8; },
                            [&](int r, int cc, float2 v) { rb[r * RS + cc] = v; });
                else
                    product(z, ra, [](int, int) { return 0; }, [](int, int) { return 8; },
                            [&](int r, int cc, float2 v) { rb[r * RS + cc].x += v.x; rb[r * RS + cc].y += v.y; });
            }
            __syncthreads();
            load_block(ra, P, P);
            __syncthreads();
            product(ra, rb, [](int, int) { return 0; }, [](int mt, int) { return 2 * mt + 2; },
                    [&](int r, int cc, float2 v) { M2[(size_t)(P + r) * Co + h * cb + cc] = make_float2(-v.x, -v.y); });
        }
    } else {
        // the neutral tile
        for (int i = tid; i < M * h; i += kCmpThreads) {
            const int j = i / h, t = i % h;
            Y2[j * Co + P + t] = make_float2(0.f, 0.f);
            W2[j * Co + P + t] = make_float2(0.f, 0.f);
        }
        for (int i = tid; i < h * P; i += kCmpThreads) M2[(size_t)(P + i / P) * Co + i % P] = make_float2(0.f, 0.f);
        for (int i = tid; i < h * h; i += kCmpThreads)
            M2[(size_t)(P + i / h) * Co + P + i % h] = make_float2(i / h == i % h ? 1.f : 0.f, 0.f);
    }
    __syncthreads();                                     // gb, gp were read from blocks that are zeroed now
    for (int i = tid; i < P * h; i += kCmpThreads) M2[(size_t)(i / h) * Co + P + i % h] = make_float2(0.f, 0.f);
    for (int j = tid; j < M; j += kCmpThreads) G2[j] = cmul(gb[j], gp[j]);
    if (turns && has) {
        const int n2 = min(h, T_ - t0 - P);
        const uint32_t *close1 = turns + (((size_t)bb * T_ + t0 + P - 1) * H + hh) * M;
        for (int i = tid; i < n2 * M; i += kCmpThreads) {
            const int t = i / M, j = i % M;
            turns[(((size_t)bb * T_ + t0 + P + t) * H + hh) * M + j] += close1[j];
        }
    }
}

template <int DK, typename T>
cudaError_t launch_fac_super(const FactorArgs &a, cudaStream_t stream, int *launches)
{
    const int sup = a.chunk / 64;
    cudaError_t e = launch_fac<DK, 64, T>(a, stream, sup);
    if (e != cudaSuccess) return e;
    if (launches) ++*launches;
    auto kern = sfda_compose_factors_kernel<DK>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)compose_smem_bytes(DK, sup - 1));
    if (e != cudaSuccess) return e;
    const int NCo = (a.T + a.chunk - 1) / a.chunk;
    for (int b = 1; b < sup; ++b) {
        kern<<<(unsigned)a.B * a.H * NCo, kCmpThreads, compose_smem_bytes(DK, b), stream>>>(a.Gamma, a.Y, a.M, a.W, a.phase_turns,
                                                                                           a.T, a.H, NCo, sup, b);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        if (launches) ++*launches;
    }
    return cudaSuccess;
}

template <typename T>
cudaError_t dispatch_fac(const FactorArgs &a, cudaStream_t s)
{
    if (a.d_k == 64 && a.chunk == 16) return launch_fac<64, 16, T>(a, s);
    if (a.d_k == 64 && a.chunk == 32) return launch_fac<64, 32, T>(a, s);
    if (a.d_k == 64 && a.chunk == 64) return launch_fac<64, 64, T>(a, s);
    if (a.d_k == 128 && a.chunk == 16) return launch_fac<128, 16, T>(a, s);
    if (a.d_k == 128 && a.chunk == 32) return launch_fac<128, 32, T>(a, s);
    if (a.d_k == 128 && a.chunk == 64) return launch_fac<128, 64, T>(a, s);
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_chunk_factors(const FactorArgs &a, cudaStream_t stream, int *launches)
{
    if (a.chunk > 64) {   // tiles of 64 tokens and their composition (needs every factor array: the tiles' Gamma wait in M)
        if ((a.chunk != 128 && a.chunk != 256) || !a.Gamma || !a.Y || !a.M || !a.W) return cudaErrorInvalidValue;
        if (a.d_k == 64) return a.dtype == 1 ? launch_fac_super<64, __nv_bfloat16>(a, stream, launches) : launch_fac_super<64, float>(a, stream, launches);
        return a.dtype == 1 ? launch_fac_super<128, __nv_bfloat16>(a, stream, launches) : launch_fac_super<128, float>(a, stream, launches);
    }
    const cudaError_t e = a.dtype == 1 ? dispatch_fac<__nv_bfloat16>(a, stream) : dispatch_fac<float>(a, stream);
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace sfda
