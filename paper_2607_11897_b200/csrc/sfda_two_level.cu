// Two-level scan over the time axis for few, long sequences.
//
// One sequence is one serial chain of chunks, so with fewer (batch, head) pairs than SMs most of the GPU idles.  The
// chunk transfer is affine in the state (Theorem "Exact affine chunk transfer"): over a time slice,
// S_out = P S_in + B with P (d_k/2 x d_k/2 complex) and B (the state the slice reaches from zero) independent of
// S_in.  So a sequence is cut into n slices that run as independent sequences:
//
//   pass 1a   every slice from a zero state (slice 0 from S_0): its B and its outputs o^(0) (final for slice 0);
//   pass 1b   every slice with v = 0 from the state [I | 0]: the first d_k/2 columns of what it reaches are P, and
//             the first d_k/2 columns of its outputs are g_t = P_t^* q_t (P_t: the transfer up to token t);
//   scan      S_1 = B_0,  S_{i+1} = P_i S_i + B_i   (n - 1 small complex products per pair);
//   correct   S_t = P_t S_in + B_t, so  S_t^* q_t = o_t^(0) + S_in^* g_t:  a [T/n x d_k/2] [d_k/2 x d_v] complex
//             product per slice and head, added to the outputs of pass 1a in place (tensor cores, bf16 operands).
//
// [B][T] is contiguous, so slice i of batch element b is simply batch element b n + i of a [B n][T / n] problem on
// the same memory: the passes are plain calls of the chunk forward.  Two chain passes, each n times as parallel,
// and a memory-bound epilogue: worth it when B H n fits the machine.  Exact algebra; P, B, g and S_in carry the
// forward's bf16 rounding once more.
#include "sfda_common.cuh"
#include "sfda_internal.h"

namespace sfda {
namespace {

constexpr int kScanThreads = 256;

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

// One CTA per (batch, head) pair and block of kScanCols value columns (the columns of a state never interact):
// S_1 = B_0 (slice 0 already started from S_0), S_{i+1} = P_i S_i + B_i; writes the initial state of every slice and
// the final state.  P_i: columns 0 .. M-1 of Pst, complex via paired rows.
constexpr int kScanCols = 16;
template <int DK, int DV>
__global__ void __launch_bounds__(kScanThreads)
two_level_scan_kernel(const float *__restrict__ Bst, const float *__restrict__ Pst, const float *__restrict__ S0,
                      float *__restrict__ Sin, float *__restrict__ S_T, int n, int H)
{
    constexpr int M = DK / 2, CT = kScanCols, RG = kScanThreads / CT, RPT = M / RG;
    static_assert(M % RG == 0 && DV % CT == 0, "row groups and column blocks must tile the state");
    __shared__ float Sr[M * CT], Si[M * CT], Pr[M * (M + 1)], Pi[M * (M + 1)];
    const int tid = threadIdx.x, bh = blockIdx.x, h = bh % H, b = bh / H, c0 = blockIdx.y * CT;
    const int c = tid % CT, g = tid / CT;
    const size_t per = (size_t)DK * DV;
    auto state = [&](const float *base, int sl) { return base + (((size_t)b * n + sl) * H + h) * per; };

    // slice 0 starts from S_0
    float *dst0 = Sin + (((size_t)b * n) * H + h) * per;
    for (int i = tid; i < DK * CT; i += kScanThreads) {
        const int row = i / CT, cc = i % CT;
        dst0[(size_t)row * DV + c0 + cc] = S0 ? S0[(size_t)bh * per + (size_t)row * DV + c0 + cc] : 0.f;
    }
    const float *B0 = state(Bst, 0);
    for (int i = tid; i < M * CT; i += kScanThreads) {
        const int j = i / CT, cc = i % CT;
        Sr[i] = B0[(size_t)(2 * j) * DV + c0 + cc];
        Si[i] = B0[(size_t)(2 * j + 1) * DV + c0 + cc];
    }
    __syncthreads();
    for (int sl = 1; sl < n; ++sl) {
        float *dst = Sin + (((size_t)b * n + sl) * H + h) * per;
        for (int i = tid; i < M * CT; i += kScanThreads) {
            const int j = i / CT, cc = i % CT;
            dst[(size_t)(2 * j) * DV + c0 + cc] = Sr[i];
            dst[(size_t)(2 * j + 1) * DV + c0 + cc] = Si[i];
        }
        const float *P = state(Pst, sl), *Bs = state(Bst, sl);
        for (int i = tid; i < M * M; i += kScanThreads) {
            const int j = i / M, l = i % M;
            Pr[j * (M + 1) + l] = P[(size_t)(2 * j) * DV + l];
            Pi[j * (M + 1) + l] = P[(size_t)(2 * j + 1) * DV + l];
        }
        __syncthreads();
        // thread = column c and a group of rows: next[j][c] = B[j][c] + sum_l P[j][l] S[l][c]
        float nr[RPT], ni[RPT];
#pragma unroll
        for (int r = 0; r < RPT; ++r) {
            const int j = g + RG * r;
            nr[r] = Bs[(size_t)(2 * j) * DV + c0 + c];
            ni[r] = Bs[(size_t)(2 * j + 1) * DV + c0 + c];
        }
        for (int l = 0; l < M; ++l) {
            const float sr = Sr[l * CT + c], si = Si[l * CT + c];
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
            Sr[j * CT + c] = nr[r];
            Si[j * CT + c] = ni[r];
        }
        __syncthreads();
    }
    if (S_T) {
        for (int i = tid; i < M * CT; i += kScanThreads) {
            const int j = i / CT, cc = i % CT;
            S_T[(size_t)bh * per + (size_t)(2 * j) * DV + c0 + cc] = Sr[i];
            S_T[(size_t)bh * per + (size_t)(2 * j + 1) * DV + c0 + cc] = Si[i];
        }
    }
}

// ---- correction o += S_in^* g on the tensor cores (mma.sync m16n8k16, bf16 operands, fp32 accumulation) -------------
// CTA = 128 tokens of one (slice, head); warp = 16 tokens x 128 channels in two halves of 64.  The A operand is the
// tile of g (tokens x 64 coordinates, Re and Im), the B operand conj(S_in) as [channel][coordinate]:
//   Re += g_re S_re + g_im S_im,   Im += g_im S_re - g_re S_im.
constexpr int kCorrThreads = 256;
constexpr int kCorrTokens = 128;
constexpr int kCorrTilesPerCta = 8;   // tiles of 128 tokens per CTA: conj(S_in) is converted once for all of them
constexpr int kCorrLd = 72;      // row stride (bf16) of the shared tiles: 144 bytes, conflict-free for ldmatrix

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const __nv_bfloat16 *p)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
__device__ __forceinline__ void ldsm_x2(uint32_t (&r)[2], const __nv_bfloat16 *p)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];"
                 : "=r"(r[0]), "=r"(r[1]) : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2])
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// g_re, g_im, o, o_im: [B n][T / n][H][128] bf16 (g: the first 64 channels);  S_in: [B n][H][128][128] float, paired rows.
__global__ void __launch_bounds__(kCorrThreads)
two_level_correct_kernel(const __nv_bfloat16 *__restrict__ g_re, const __nv_bfloat16 *__restrict__ g_im,
                         const float *__restrict__ S_in, __nv_bfloat16 *__restrict__ o, __nv_bfloat16 *__restrict__ o_im,
                         int Ts, int H, int n)
{
    constexpr int DV = 128, MC = 64;
    const int bq = blockIdx.z, h = blockIdx.y;
    if (bq % n == 0) return;                        // slice 0 started from the true initial state already
    extern __shared__ __align__(16) unsigned char corr_smem[];
    __nv_bfloat16 *Are = reinterpret_cast<__nv_bfloat16 *>(corr_smem);       // [128 tokens][kCorrLd]
    __nv_bfloat16 *Aim = Are + kCorrTokens * kCorrLd;
    __nv_bfloat16 *Bre = Aim + kCorrTokens * kCorrLd;                        // [128 channels][kCorrLd]: S_in^T
    __nv_bfloat16 *Bim = Bre + DV * kCorrLd;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // S_in^T as bf16, once per CTA: element (channel c, coordinate l) = S_in[l][c]; consecutive threads take
    // consecutive channels
    const float *Sp = S_in + ((size_t)bq * H + h) * (2 * MC) * DV;
    for (int idx = tid; idx < MC * DV; idx += kCorrThreads) {
        const int l = idx / DV, c = idx % DV;
        Bre[c * kCorrLd + l] = __float2bfloat16_rn(Sp[(size_t)(2 * l) * DV + c]);
        Bim[c * kCorrLd + l] = __float2bfloat16_rn(Sp[(size_t)(2 * l + 1) * DV + c]);
    }
    const int arow = 16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1), acol = 8 * (lane >> 4);   // ldmatrix x4 addresses
    const int brow = lane & 7, bcol = 8 * ((lane >> 3) & 1);                                     // ldmatrix x2
    const int gq = lane >> 2, tg = lane & 3;
    // this CTA's tiles of 128 tokens
#pragma unroll 1
    for (int tile = blockIdx.x * kCorrTilesPerCta; tile < (blockIdx.x + 1) * kCorrTilesPerCta; ++tile) {
    const int t0 = tile * kCorrTokens;
    if (t0 >= Ts) break;
    const int rows = min(kCorrTokens, Ts - t0);

    // g tile: 128 rows of 128 bytes (Re and Im), 16 bytes per copy; rows past the slice are zero
    for (int idx = tid; idx < kCorrTokens * 8; idx += kCorrThreads) {
        const int r = idx >> 3, ch = idx & 7;
        const size_t src = (((size_t)bq * Ts + t0 + r) * H + h) * DV + 8 * ch;
        uint4 vr = make_uint4(0u, 0u, 0u, 0u), vi = vr;
        if (r < rows) {
            vr = *reinterpret_cast<const uint4 *>(g_re + src);
            vi = *reinterpret_cast<const uint4 *>(g_im + src);
        }
        *reinterpret_cast<uint4 *>(Are + r * kCorrLd + 8 * ch) = vr;
        *reinterpret_cast<uint4 *>(Aim + r * kCorrLd + 8 * ch) = vi;
    }
    __syncthreads();

    // Corrections of one half of the channels as bf16 [128 tokens][64 channels] (Re, then Im) behind the operand
    // tiles, so that the read-modify-write of the outputs runs on whole 16-byte pieces of a row with every load of a
    // thread in flight at once.
    constexpr int kDLd = 64 + 8;
    __nv_bfloat16 *Dre = Bim + DV * kCorrLd, *Dim = Dre + kCorrTokens * kDLd;
    constexpr int kPieces = kCorrTokens * 8 / kCorrThreads;              // 16-byte pieces per thread, plane and half
#pragma unroll 1
    for (int half = 0; half < 2; ++half) {
        float dre[8][4], dim[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int x = 0; x < 4; ++x) dre[nt][x] = dim[nt][x] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            uint32_t are[4], aim[4], aren[4];
            ldsm_x4(are, Are + arow * kCorrLd + 16 * ks + acol);
            ldsm_x4(aim, Aim + arow * kCorrLd + 16 * ks + acol);
#pragma unroll
            for (int x = 0; x < 4; ++x) aren[x] = are[x] ^ 0x80008000u;      // -g_re
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                uint32_t bre[2], bim[2];
                const int c = 64 * half + 8 * nt + brow;
                ldsm_x2(bre, Bre + c * kCorrLd + 16 * ks + bcol);
                ldsm_x2(bim, Bim + c * kCorrLd + 16 * ks + bcol);
                mma_bf16(dre[nt], are, bre);
                mma_bf16(dre[nt], aim, bim);
                mma_bf16(dim[nt], aim, bre);
                mma_bf16(dim[nt], aren, bim);
            }
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int hr = 0; hr < 2; ++hr) {
                const int r = 16 * warp + gq + 8 * hr, c = 8 * nt + 2 * tg;
                *reinterpret_cast<__nv_bfloat162 *>(Dre + r * kDLd + c) = __floats2bfloat162_rn(dre[nt][2 * hr], dre[nt][2 * hr + 1]);
                *reinterpret_cast<__nv_bfloat162 *>(Dim + r * kDLd + c) = __floats2bfloat162_rn(dim[nt][2 * hr], dim[nt][2 * hr + 1]);
            }
        __syncthreads();
        auto add_plane = [&](__nv_bfloat16 *dst, const __nv_bfloat16 *D) {
            uint4 cur[kPieces];
#pragma unroll
            for (int x = 0; x < kPieces; ++x) {
                const int idx = tid + x * kCorrThreads, r = idx >> 3, ch = idx & 7;
                cur[x] = make_uint4(0u, 0u, 0u, 0u);
                if (r < rows)
                    cur[x] = *reinterpret_cast<const uint4 *>(dst + (((size_t)bq * Ts + t0 + r) * H + h) * DV + 64 * half + 8 * ch);
            }
#pragma unroll
            for (int x = 0; x < kPieces; ++x) {
                const int idx = tid + x * kCorrThreads, r = idx >> 3, ch = idx & 7;
                if (r >= rows) continue;
                const uint4 dl = *reinterpret_cast<const uint4 *>(D + r * kDLd + 8 * ch);
                const uint32_t *pc = reinterpret_cast<const uint32_t *>(&cur[x]), *pd = reinterpret_cast<const uint32_t *>(&dl);
                uint32_t out[4];
#pragma unroll
                for (int y = 0; y < 4; ++y) {
                    const float2 a2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&pc[y]));
                    const float2 b2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&pd[y]));
                    const __nv_bfloat162 sum = __floats2bfloat162_rn(a2.x + b2.x, a2.y + b2.y);
                    out[y] = *reinterpret_cast<const uint32_t *>(&sum);
                }
                *reinterpret_cast<uint4 *>(dst + (((size_t)bq * Ts + t0 + r) * H + h) * DV + 64 * half + 8 * ch) =
                    make_uint4(out[0], out[1], out[2], out[3]);
            }
        };
        add_plane(o, Dre);
        if (o_im) add_plane(o_im, Dim);
        __syncthreads();                           // the next half overwrites the corrections
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
// of pass 1a, B, [I | 0], P, true initial states), a zero v and the outputs of pass 1b (Re and Im: g).
size_t forward_two_level_bytes(const ForwardArgs &a, int n)
{
    const size_t states = (size_t)a.B * n * a.H * a.d_k * a.d_v * 4;
    const size_t tokens = (size_t)a.B * a.T * a.H * a.d_v * 2;
    return round256(forward_ws_scratch_bytes(a.B * n, a.H)) + 5 * round256(states) + 3 * round256(tokens);
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
    void *g_re = w;                                     w += tokens;
    void *g_im = w;

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
    // pass 1a: B of every slice and the outputs from a zero state (slice 0 from S_0: its outputs are final)
    s.S0 = S_a; s.S_T = B_st;
    if ((e = launch_forward_ws(s, fwd_ws, fwd_bytes, stream, launches)) != cudaSuccess) return e;
    // pass 1b: P of every slice, and g_t = P_t^* q_t in the first d_k / 2 channels of its outputs
    // (same scratch block: the status word keeps a timeout of pass 1a, so that the caller's one read sees either)
    s.v = v_zero; s.S0 = S_id; s.S_T = P_st; s.o = g_re; s.o_im = g_im;
    if ((e = launch_forward_ws(s, fwd_ws, fwd_bytes, stream, launches, false)) != cudaSuccess) return e;
    // scan over the slices
    two_level_scan_kernel<128, 128><<<dim3((unsigned)(a.B * a.H), 128 / kScanCols), kScanThreads, 0, stream>>>(
        B_st, P_st, a.S0, S_in, a.S_T, n, a.H);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (launches) ++*launches;
    // correction: o += S_in^* g for every slice but the first
    const size_t csmem = (size_t)((2 * kCorrTokens + 2 * 128) * kCorrLd + 2 * kCorrTokens * (64 + 8)) * 2;
    if ((e = cudaFuncSetAttribute(two_level_correct_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)csmem)) != cudaSuccess)
        return e;
    const int ctiles = (s.T + kCorrTokens - 1) / kCorrTokens;
    const dim3 cgrid((unsigned)((ctiles + kCorrTilesPerCta - 1) / kCorrTilesPerCta), (unsigned)a.H, (unsigned)(a.B * n));
    two_level_correct_kernel<<<cgrid, kCorrThreads, csmem, stream>>>(
        static_cast<const __nv_bfloat16 *>(g_re), static_cast<const __nv_bfloat16 *>(g_im), S_in,
        static_cast<__nv_bfloat16 *>(a.o), static_cast<__nv_bfloat16 *>(a.o_im), s.T, a.H, n);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (launches) ++*launches;
    return cudaSuccess;
}

}  // namespace sfda
