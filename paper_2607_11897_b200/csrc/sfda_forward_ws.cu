// Warp-specialised tensor-core chunk-WY forward for sm_100a: bf16 q/k/v, d_k = d_v = 128, chunk C = 64.
//
// One persistent CTA per SM walks a stream of work units (a unit = one time slice of one (batch, head) sequence;
// the boundary state between slices goes through the caller's workspace).  Four roles run concurrently on
// different chunks and hand tiles to one another through mbarriers:
//
//   PREP  (8 warps)  chunk j+1: cumulative phase-decay gamma_t = a_t e^{i phi_t} (Eq. "constructive-Gamma": scan
//                    partials per token octet, then a running complex product token by token), rotated/decayed
//                    operand tiles in shared memory; it also reads the finished outputs of chunk j-1 out of
//                    tensor memory for the TMA store.
//   SOLVE (4 warps)  chunk j+1: drains the Gram blocks from tensor memory, inverts the unit-lower WY system
//                    (Eq. "constructive-M": M = (I + L)^{-1}) by 8x8 blocks and tensor-core merges, writes the
//                    M_beta and Aq tiles.
//   CHAIN (8 warps)  chunk j: the state-dependent conversions between the tcgen05 products
//                    (state pass, R = V - W^* S_0, E); they own the TMEM <-> register traffic of the chain.
//   CTRL  (4 warps)  issue every tcgen05.mma / commit, the TMA copies and the L2 prefetch of the inputs.
//
// The per-chunk code of all roles has to stay small: the SM's instruction cache holds about 32 KB, and what does
// not fit is fetched from the GPC-level cache chunk after chunk.  Hence the rolled loops with run-time operand
// selection, the single call sites, and the absence of integer divisions and of generic-address arithmetic below.
//
// Algebra (k'_t = e^{-i phi_t} k_t, q'_t = e^{-i phi_t} q_t, all tiles bf16, de-interleaved [Re | Im]):
//   W_t = a_t k'_t (= conj(gamma_t) k_t, Eq. "constructive-W"),  Qt_t = a_t q'_t,  Kc_t = k'_t / a_t
//   Kt[t][i] = W_t^* Kc_i (i < t),  Aq[t][i] = Qt_t^* Kc_i (i <= t)
//   M_beta = (I + D_beta Kt)^{-1} D_beta,  R = V - W^* S_0,  E = M_beta R            (Eq. "apply-transfer")
//   rho_t = Qt_t^* S_0 + sum_{i<=t} Aq[t][i] e_i^T,  o_t = conj(rho_t)               (Thm "Prefix outputs")
//   S_C = e^{i phi_C} a_C (S_0 + sum_t Kc_t e_t^T)                                    (boundary-state scan)
// The fp32 state lives in tensor memory, transposed (lane = value channel, column = key channel
// [Re j | Im j]); the update accumulates onto the unscaled S_0 and the factor e^{i phi_C} a_C is applied by
// the next chunk's state pass, so no operand depends on the chunk's total decay.
#include <cuda.h>

#include <mutex>

#include "sfda_common.cuh"
#include "sfda_internal.h"
#include "sfda_tc_ptx.cuh"

namespace sfda {
namespace {

using namespace tc;

constexpr int C = 64, DK = 128, DV = 128, M = 64;
constexpr int kChainWarps = 8, kSolveWarps = 4, kPrepWarps = 8;
constexpr int kCtrlWarps = 4;   // a full warpgroup, so that it can hand its registers to the others; one thread works
constexpr int kThreads = 32 * (kChainWarps + kSolveWarps + kPrepWarps + kCtrlWarps);   // 768
constexpr int kChainThreads = 32 * kChainWarps, kSolveThreads = 32 * kSolveWarps, kPrepThreads = 32 * kPrepWarps;
// The CTA is launched with 80 registers per thread (768 * 80 = 61440); the working roles take what CTRL gives up:
// (8 + 4 + 8) * 88 + 4 * 40 = 1920 warp rows = 61440 registers.
constexpr int kRegsWork = 88, kRegsCtrl = 40;
constexpr int kTB = 2;
            // tokens per trip of PREP's operand loop

// ---- shared memory map (bytes from a 1024-aligned base) -------------------------------------------------
constexpr int kTile = 8192;                       // 64 rows x 128 B, 128B swizzle
constexpr int OFF_WQ = 0;                         // [2 slots][re | im][128 rows: W then Qt], K-major     64 KB
constexpr int OFF_KC = OFF_WQ + 2 * 4 * kTile;    // [2 slots] Kc [t][j], re | im: K-major B of the Gram, 32 KB
                                                  //           MN-major B of the state update
constexpr int OFF_MB = OFF_KC + 2 * 2 * kTile;    // M_beta [t][i], re | im                                16 KB
constexpr int OFF_AQ = OFF_MB + 2 * kTile;        // [2 slots] Aq [t][i], re | im; also stages o_im        32 KB
constexpr int OFF_V = OFF_AQ + 2 * 2 * kTile;     // v staging [t][128] bf16 (TMA load)                    16 KB
constexpr int OFF_OST = OFF_V + 16384;            // o staging [t][128] bf16 (TMA store)                   16 KB
constexpr int LS = 68;                            // row stride (floats) of the solve scratch
constexpr int OFF_LX = OFF_OST + 16384;           // L -> X in place, fp32 [64][LS], re | im               34 KB
constexpr int OFF_MISC = OFF_LX + 2 * 64 * LS * 4;
constexpr int kMiscBytes = 13312;
constexpr int kSmemBytes = OFF_MISC + kMiscBytes + 1024;   // + slack for the 1024-byte alignment
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA exceeded");

enum Bar {
    B_PREP_FULL0, B_PREP_FULL1,     // PREP -> CTRL: W/Qt/Kc tiles of the slot are written
    B_STORE_DONE0, B_STORE_DONE1,   // CTRL: the output store of a chunk of this parity has read its staging
    B_GRAM_FULL, B_GRAM_DRAINED,    // commit / SOLVE: one Gram half is in tensor memory / has been read out
    B_MB_FULL, B_AQ_FULL0, B_AQ_FULL1,
    B_D1_DONE, B_O1_DONE, B_E_DONE, B_UPD_DONE,
    B_S16_A, B_S16_B, B_R16_A, B_R16_B, B_E16_A, B_E16_B,   // first / second half of a bf16 operand is written
    B_O_STAGED,
    B_V_FULL,
    B_NORM_FULL,                    // SOLVE -> CHAIN (fused front end): the chunk's key scales are written
    kNumBars
};

// One chunk of a CTA's stream of chunks (see ChunkCursor below).
struct __align__(16) ChunkInfo {
    int b, h, bh, jg;           // sequence, chunk index inside the sequence
    uint32_t want;              // arrivals at the sequence's counter that the piece waits for (unless seq_first)
    bool first;                 // first chunk of its piece
    bool seq_first, seq_last;   // the piece starts / ends its sequence
    bool pad_;
    int pad2_[2];
};
static_assert(sizeof(ChunkInfo) == 32, "ring entries are copied as two 16-byte words");
constexpr int kRing = 8;        // chunks whose description is kept (the roles are at most a few chunks apart)

struct Misc {
    float part_lg[2][8][M];                 // per-group partial products / phase sums, two chunks deep
    uint32_t part_turns[2][8][M];
    float close_re[4][M], close_im[4][M];   // a_C e^{i phi_C} of a ring of four chunks, real and imaginary parts
    float beta[4][C];
    float kscale[4][C];                     // fused front end: 1 / (|k_raw| + eps) per token, ring of four chunks
    uint4 cursor_raw[3];                    // the prologue's cursor (a ChunkCursor), taken over by PREP
    ChunkInfo ring[kRing];                  // description of chunk j at ring[j % kRing], published by PREP two chunks ahead
    unsigned long long bars[kNumBars];
    uint32_t tmem_base;
    uint32_t wait_limit;                    // SM-clock ticks after which a wait gives up
    volatile int abort;
};
static_assert(sizeof(Misc) <= kMiscBytes, "misc area too small");

// ---- tensor memory map (columns) ----------------------------------------------------------------------
constexpr uint32_t TM_S32 = 0;      // state fp32 [Re j | Im j]
constexpr uint32_t TM_X16 = 128;    // bf16 A operand: S_0, then R, then E (64 packed columns)
constexpr uint32_t TM_GRAM = 192;   // Gram half (Re, then Im): lanes 0..63 Kt rows, 64..127 Aq rows
constexpr uint32_t TM_ACC = 256;    // [D1/E re | rho re | D1/E im | rho im], 64 columns each

struct Params {
    const __nv_bfloat16 *q, *k;
    const float *alpha, *theta, *beta, *S0;
    float *S_T;
    uint32_t *phase_out; // [B*H][NC][64] chunk-closing phase in 2^-32 turns, or nullptr (plain instantiation only)
    uint32_t *status;
    uint32_t *flags;     // [B*H] arrival counters of the pieces of a cut sequence (only used when sequences are cut)
    float *handoff;      // [B*H][d_k][d_v] boundary states between the pieces (only used when sequences are cut)
    int T, H, has_o_im;
    uint32_t wait_limit;   // ticks of the SM clock after which a device-side wait gives up
    int withhold;          // diagnostic launches only: boundary states are written but never announced
    int BH, U, Q, n_units;   // sequences, chunks per work unit, time slices per sequence, Q * BH
    int bal, NC, bal_base, bal_rem;   // balanced partition: on / off, chunks per sequence, BH * NC = grid * base + rem
    uint32_t magic_BH, magic_H, magic_NC;   // floor(2^32 / d) + 1 (0 for d = 1): quotients by multiplication
    // fused stable parameterisation (only read by the kFused instantiation): alpha = a_lo + a_range sigmoid(a),
    // theta = th_max tanh(b), beta = sigmoid(c), k = k_raw / (|k_raw| + eps)
    float a_lo, a_range, th_max, th_m2, eps;   // th_m2 = -2 th_max
};

// Tensor maps of the arrays the copy engine touches: [B][T][H][128] bf16 (v, o, o_im, q, k) or [B][T][H][64] fp32
// (alpha, theta), box = 64 tokens of one head.
struct Maps {
    CUtensorMap v, o, oim, q, k, al, th;
};

// Work units, in one of two partitions chosen by the launcher.
// Sliced: a sequence is cut into Q time slices of U chunks; unit u = slice * BH + sequence; CTA c works through
// units c, c + gridDim, ...  Units are handed out in increasing order, so the unit a CTA waits for is always already
// running or done.
// Balanced (only with at least as many sequences as CTAs): the B*H*NC chunks of all sequences, laid end to end,
// are cut into gridDim contiguous ranges of equal length (to within one chunk), so a range holds whole sequences
// plus the tail of one sequence at its start and the head of another at its end, and a sequence is cut at most
// once.  A CTA takes the pieces of its range in DESCENDING sequence order: the head piece first, which the next
// CTA needs only for the piece it takes last.
// Either way a CTA's pieces form ONE stream of chunks, so its pipeline never drains between them; only the state
// pass notices a boundary (it writes the finished state out and takes the next one in).  A piece that does not
// start its sequence begins from the boundary state its predecessor left in `handoff`; its CTA waits for that
// (bounded).  All CTAs are resident (cooperative launch).
// Walks the stream chunk by chunk; the quotients are taken once per piece, not once per chunk.
struct ChunkCursor {
    ChunkInfo ci;
    int j_end, u;   // chunk index at which the piece ends; unit index (sliced) or first chunk of the range (balanced)
    // n / d for n * d < 2^32 from the precomputed floor(2^32 / d) + 1 (d = 1 is flagged by 0)
    static __device__ __forceinline__ int quot(int n, uint32_t magic) { return magic ? (int)__umulhi((uint32_t)n, magic) : n; }
    // this CTA's range of the balanced partition: [lo, lo + n)
    static __device__ __forceinline__ void range(const Params &p, int &lo, int &n)
    {
        const int c = (int)blockIdx.x;
        lo = c * p.bal_base + min(c, p.bal_rem);
        n = p.bal_base + (c < p.bal_rem ? 1 : 0);
    }
    static __device__ __forceinline__ int stream_chunks(const Params &p)
    {
        if (p.bal) {
            int lo, n;
            range(p, lo, n);
            return n;
        }
        return ((p.n_units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x) * p.U;
    }
    __device__ __forceinline__ void set_piece(const Params &p)
    {
        if (p.bal) {
            ci.jg = max(u - ci.bh * p.NC, 0);
            ci.seq_first = ci.jg == 0;
            ci.want = 8u;
        } else {
            const int q = quot(u, p.magic_BH);
            ci.bh = u - q * p.BH;
            ci.jg = q * p.U;
            j_end = ci.jg + p.U;
            ci.seq_first = q == 0;
            ci.seq_last = q == p.Q - 1;
            ci.want = 8u * (uint32_t)q;
        }
        ci.b = quot(ci.bh, p.magic_H);
        ci.h = ci.bh - ci.b * p.H;
        ci.first = true;
    }
    ChunkCursor() = default;
    // hand-over through shared memory (three 16-byte words)
    __device__ __forceinline__ void store(uint4 *dst) const
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(this);
        dst[0] = src[0]; dst[1] = src[1]; dst[2] = src[2];
    }
    static __device__ __forceinline__ ChunkCursor load(const uint4 *src)
    {
        ChunkCursor c;
        uint4 *dst = reinterpret_cast<uint4 *>(&c);
        dst[0] = src[0]; dst[1] = src[1]; dst[2] = src[2];
        return c;
    }
    __device__ __forceinline__ explicit ChunkCursor(const Params &p) : u((int)blockIdx.x)
    {
        if (p.bal) {
            int n;
            range(p, u, n);
            ci.bh = quot(u + n - 1, p.magic_NC);
            j_end = u + n - ci.bh * p.NC;
            ci.seq_last = j_end == p.NC;
        }
        set_piece(p);
    }
    __device__ __forceinline__ void next(const Params &p)
    {
        ci.first = false;
        if (++ci.jg == j_end) {
            if (p.bal) {
                --ci.bh;
                j_end = p.NC;
                ci.seq_last = true;
            } else {
                u += (int)gridDim.x;
            }
            set_piece(p);
        }
    }
};

// The chunks' descriptions go through a small ring in shared memory: ONE thread (of PREP) walks the cursor, two
// chunks ahead of PREP's own work, and every role reads chunk j's entry after an event that is ordered behind its
// publication (the start of the kernel for chunks 0 and 1; for chunk j >= 2 the tiles of chunk j - 2, which PREP
// announces after publishing).  That keeps the cursor's code out of the other roles' loops.
__device__ __forceinline__ void ring_put(Misc &mi, int j, const ChunkInfo &ci)
{
    const uint4 *src = reinterpret_cast<const uint4 *>(&ci);
    uint4 *dst = reinterpret_cast<uint4 *>(&mi.ring[j & (kRing - 1)]);
    dst[0] = src[0];
    dst[1] = src[1];
}
__device__ __forceinline__ ChunkInfo ring_get(const Misc &mi, int j)
{
    ChunkInfo ci;
    const uint4 *src = reinterpret_cast<const uint4 *>(&mi.ring[j & (kRing - 1)]);
    reinterpret_cast<uint4 *>(&ci)[0] = src[0];
    reinterpret_cast<uint4 *>(&ci)[1] = src[1];
    return ci;
}

static_assert(sizeof(ChunkCursor) == 48, "the cursor is handed over as three 16-byte words");

// Development builds only (-DSFDA_WS_CHAOS): a pseudo-random pause of 0.1 to 1.1 us after one in eight barrier
// arrivals and completed waits.  The results do not depend on timing, so a build with the pauses must reproduce
// the plain build bit for bit; an ordering hazard between the roles shows as a difference.
#ifdef SFDA_WS_CHAOS
__device__ __forceinline__ void chaos(uint32_t salt)
{
    uint32_t x = (uint32_t)clock() * 2654435761u + salt * 40503u + (threadIdx.x >> 5) * 9176u;
    x ^= x >> 13; x *= 0x5bd1e995u; x ^= x >> 15;
    if ((x & 7u) == 0u) __nanosleep(100u + ((x >> 8) & 1023u));
}
#else
__device__ __forceinline__ void chaos(uint32_t) {}
#endif
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One arrival per warp: the warp's lanes order their writes among themselves with __syncwarp, then one lane
// arrives (a barrier counted in warps completes after a handful of shared-memory atomics instead of hundreds).
__device__ __forceinline__ void warp_arrive(unsigned long long *bar)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
#ifdef SFDA_WS_CHAOS
    __syncwarp();
    chaos((uint32_t)(size_t)bar);
    __syncwarp();
#endif
}
template <int N>
__device__ __forceinline__ void regs_inc()
{
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void regs_dec()
{
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
// Barrier among the threads of one role (hardware barrier `id`); returns the OR of `flag` over the role.
__device__ __forceinline__ bool role_sync_or(int id, int nthreads, bool flag)
{
    uint32_t out;
    asm volatile(
        "{\n.reg .pred p, q;\nsetp.ne.b32 q, %3, 0;\nbarrier.cta.red.or.pred p, %1, %2, q;\nselp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(out)
        : "r"(id), "r"(nthreads), "r"((uint32_t)flag)
        : "memory");
    return out != 0;
}
__device__ __forceinline__ void role_sync(int id, int nthreads)
{
    asm volatile("barrier.cta.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}


// Wait for completion number k of a barrier; gives up after the launch's wait limit (about a second: 2^31 ticks of
// the SM clock, unless the caller asked for less) or as soon as any other wait of the CTA has given up, and raises
// the abort flag.  try_wait parks the thread in hardware for up to the hinted time, so waiting warps do
// not compete with working ones for issue slots.  Kept to a handful of instructions: it is inlined at every
// wait, and the kernel's per-chunk code has to stay inside the SM's instruction cache.
template <bool kDiag>
__device__ __forceinline__ bool wait_k(Misc &mi, int bar, int k)
{
    const uint32_t addr = smem_u32(&mi.bars[bar]), parity = (uint32_t)k & 1u;
    const uint32_t t0 = (uint32_t)clock();
    do {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok)
            : "r"(addr), "r"(parity), "r"(20000u)
            : "memory");
        if (ok) {
            chaos(addr + 77u);
            return true;
        }
        // the diagnostic instantiation takes its limit from the launch and also leaves as soon as any other wait
        // of the CTA has given up (a few more instructions per wait than the product kernel can afford)
    } while (kDiag ? (!mi.abort && (uint32_t)clock() - t0 < mi.wait_limit) : ((uint32_t)clock() - t0 < 0x80000000u));
    mi.abort = 1;
    return false;
}

// ---- CTRL: three warps issue all tensor-core and TMA work ------------------------------------------------
// A CTRL warp runs its loop with all 32 lanes converged and elects one lane only around the instructions that
// a single thread must issue.  (Issued from inside a one-thread branch, every tensor-core instruction costs some
// thirty instructions that move its operands into uniform registers; from converged code it costs about five.)
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}\n" : "=r"(pred));
    return pred != 0;
}
// wait_k with a warp-uniform outcome, so that a warp leaves (or stays) as a whole
template <bool kDiag>
__device__ __forceinline__ bool wait_k_warp(Misc &mi, int bar, int k)
{
    return __all_sync(0xffffffffu, wait_k<kDiag>(mi, bar, k) ? 1 : 0) != 0;
}

// One complex product as four real ones (g = 0..3), each of four K = 16 instructions:
//   Re += x_re b_re,  Re -+= x_im b_im,  Im += x_im b_re,  Im +-= x_re b_im
// A (x) is the bf16 operand in tensor memory (or, for the Gram, tiles in shared memory); `a_im`, `b_im`, `d_im`
// are the imaginary parts' addresses; kNegMask has bit g set for the products that are subtracted; `fresh`:
// the accumulators start from zero.  `b_step`: descriptor advance of B per K = 16 (2 for a K-major tile,
// 128 for an MN-major one).  The state update uses the same products with conj(E)-side roles swapped, which
// `swap` selects: Re += x_re b_re, Re -= x_im b_im, Im += x_re b_im, Im += x_im b_re.
// `part` selects the products of one accumulator: 0 = Re (g = 0, 1), 1 = Im (g = 2, 3), 2 = both.  The two halves
// touch different accumulator columns, so two threads can issue them side by side (instructions of one thread
// execute in order, which the accumulation inside a half needs; nothing orders two threads, nor has to).
// kMask: the K = 16 steps to issue (bit ks); the operands arrive in two halves, and the steps that only need the
// first half go out while the second is still being written.  With kFresh the lowest step of the mask starts the
// accumulators from zero (so the call with kFresh has to be the first for its accumulators).
template <int kNegMask, bool kFresh, bool kSwap, uint32_t kBStep, int kMask = 15>
__device__ __forceinline__ void issue_complex(uint32_t d_re, uint32_t d_im, uint32_t a_re, uint32_t a_im, uint32_t b_re,
                                              uint32_t b_im, uint32_t dhi, uint32_t id, int part)
{
    if (elect_one()) {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            if (part != 2 && (g >> 1) != part) continue;
            const bool odd = g & 1, mid = g == 1 || g == 2;
            const uint32_t d = g < 2 ? d_re : d_im;
            const uint32_t a = (kSwap ? odd : mid) ? a_im : a_re;
            const uint32_t b = (kSwap ? mid : odd) ? b_im : b_re;
            const uint32_t idg = id | ((kNegMask >> g & 1) ? 1u << 14 : 0u);
            constexpr int kFirst = (kMask & 1) ? 0 : (kMask & 2) ? 1 : (kMask & 4) ? 2 : 3;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
                if (kMask >> ks & 1)
                    mma_ts2(d, a + 8 * ks, b + kBStep * ks, dhi, idg, (!kFresh || odd || ks != kFirst) ? 1u : 0u);
        }
    }
    __syncwarp();
}

// ---- input prefetch ------------------------------------------------------------------------------------
// PREP reads q, k, alpha, theta straight from global memory (no shared memory is left to stage them).  So that
// those loads find their lines in L2 instead of stalling on HBM, the copy engine is asked to bring the four tiles
// of a chunk into L2 two chunks before PREP gets there: four instructions per chunk.
__device__ __forceinline__ void tma_prefetch_4d(const CUtensorMap *map, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}
__device__ __forceinline__ void prefetch_chunk(const Maps &maps, const ChunkInfo &ci)   // one thread
{
    tma_prefetch_4d(&maps.al, 0, ci.h, ci.jg * C, ci.b);
    tma_prefetch_4d(&maps.th, 0, ci.h, ci.jg * C, ci.b);
    tma_prefetch_4d(&maps.k, 0, ci.h, ci.jg * C, ci.b);
    tma_prefetch_4d(&maps.q, 0, ci.h, ci.jg * C, ci.b);
}

// The issuing work is split over four warps (they sit on different schedulers):
//   roles 0, 3  the products on the state's dependency chain: D1, rho_1, E, the state update; role 0 issues the
//               products into the real accumulators, role 3 those into the imaginary ones (issuing, not the
//               tensor pipe, is what takes the time: about a hundred cycles per instruction)
//   role 1      the output product rho += Aq E and the output stores
//   role 2      the v loads, the Gram products (they run ahead of the chain) and the L2 prefetch of the inputs
template <bool kDiag>
__device__ __forceinline__ void run_ctrl(int role, uint8_t *smem, Misc &mi, uint32_t tmem, const Maps &maps,
                                         const Params &p, int n_chunks)
{
    const CUtensorMap *tm_v = &maps.v, *tm_o = &maps.o, *tm_oim = &maps.oim;
    const uint64_t dbase = smem_desc(smem_u32(smem));                     // descriptor of byte offset 0
    const uint32_t dlo = (uint32_t)dbase, dhi = (uint32_t)(dbase >> 32);
    unsigned long long *bars = mi.bars;
    constexpr uint32_t I64 = idesc(64, 0), I64M = idesc(64, 0) | (1u << 16);   // M: B MN-major
    constexpr uint32_t kIm = kTile >> 4;                                  // re -> im tile, in descriptor units
    const uint32_t x_re = tmem + TM_X16, acc = tmem + TM_ACC;
    const uint32_t m_re = dlo + (OFF_MB >> 4);

    if (role == 0 || role == 3) {
        const int part = role == 0 ? 0 : 1;      // this warp's accumulator half
#pragma unroll 1
        for (int j = 0; j < n_chunks; ++j) {
            const int s = j & 1, u = j >> 1;
            const uint32_t w_re = dlo + ((OFF_WQ + s * 4 * kTile) >> 4), k_re = dlo + ((OFF_KC + s * 2 * kTile) >> 4);
            // -D1 = -W^* S_0 (all four real products with the opposite sign, so that R = V + (-D1) needs no multiplication
            // on the way to the operand columns) as soon as S_0 is there; rho_1 = Qt^* S_0 (the Qt rows follow the W rows in the slot's
            // tiles) once rho of the previous chunk has been read out.  Both read S_0 from the operand columns.
            // (the state pass writes S_0 in two halves: key coordinates 0-15 and 32-47 = k-steps 0 and 2 first)
            if (!wait_k_warp<kDiag>(mi, B_S16_A, j)) return;
            if (!wait_k_warp<kDiag>(mi, B_PREP_FULL0 + s, u)) return;
            tc_fence_after();
            issue_complex<7, true, false, 2, 5>(acc, acc + 128, x_re, x_re + 32, w_re, w_re + 2 * kIm, dhi, I64, part);
            if (!wait_k_warp<kDiag>(mi, B_S16_B, j)) return;
            tc_fence_after();
            issue_complex<7, false, false, 2, 10>(acc, acc + 128, x_re, x_re + 32, w_re, w_re + 2 * kIm, dhi, I64, part);
            if (elect_one()) mma_commit(&bars[B_D1_DONE]);
            if (j > 0 && !wait_k_warp<kDiag>(mi, B_O_STAGED, j - 1)) return;
            tc_fence_after();
            issue_complex<8, true, false, 2>(acc + 64, acc + 192, x_re, x_re + 32, w_re + kIm, w_re + 3 * kIm, dhi, I64, part);
            if (elect_one()) {
                mma_commit(&bars[B_O1_DONE]);
            }
            // E = M_beta R (R arrives in two halves of 32 tokens = two k-steps each)
            if (!wait_k_warp<kDiag>(mi, B_R16_A, j)) return;
            if (!wait_k_warp<kDiag>(mi, B_MB_FULL, j)) return;
            tc_fence_after();
            issue_complex<2, true, false, 2, 3>(acc, acc + 128, x_re, x_re + 32, m_re, m_re + kIm, dhi, I64, part);
            if (!wait_k_warp<kDiag>(mi, B_R16_B, j)) return;
            tc_fence_after();
            issue_complex<2, false, false, 2, 12>(acc, acc + 128, x_re, x_re + 32, m_re, m_re + kIm, dhi, I64, part);
            if (elect_one()) mma_commit(&bars[B_E_DONE]);
            // S += E^T Kc (Kc as MN-major B: rows = tokens)
            if (!wait_k_warp<kDiag>(mi, B_E16_A, j)) return;
            tc_fence_after();
            issue_complex<2, false, true, 128, 3>(tmem + TM_S32, tmem + TM_S32 + 64, x_re, x_re + 32, k_re, k_re + kIm, dhi, I64M, part);
            if (!wait_k_warp<kDiag>(mi, B_E16_B, j)) return;
            tc_fence_after();
            issue_complex<2, false, true, 128, 12>(tmem + TM_S32, tmem + TM_S32 + 64, x_re, x_re + 32, k_re, k_re + kIm, dhi, I64M, part);
            if (elect_one()) {
                mma_commit(&bars[B_UPD_DONE]);
            }
        }
    } else if (role == 1) {
        // iteration j: store the outputs of chunk j - 1 (once staged), then issue rho += Aq E of chunk j
#pragma unroll 1
        for (int j = 0; j <= n_chunks; ++j) {
            if (j > 0) {
                if (!wait_k_warp<kDiag>(mi, B_O_STAGED, j - 1)) return;
                const ChunkInfo pc = ring_get(mi, j - 1);
                if (elect_one()) {
                    tma_store_4d(tm_o, smem + OFF_OST, 0, pc.h, pc.jg * C, pc.b);
                    tma_store_4d(tm_o, smem + OFF_OST + kTile, 64, pc.h, pc.jg * C, pc.b);
                    if (p.has_o_im) {
                        const uint8_t *src = smem + OFF_AQ + ((j - 1) & 1) * 2 * kTile;
                        tma_store_4d(tm_oim, src, 0, pc.h, pc.jg * C, pc.b);
                        tma_store_4d(tm_oim, src + kTile, 64, pc.h, pc.jg * C, pc.b);
                    }
                    tma_store_commit();
                    if (j < n_chunks) {
                        tma_store_wait_read();
                        mbar_arrive(&bars[B_STORE_DONE0 + ((j - 1) & 1)]);
                    } else {
                        tma_store_wait_all();
                    }
                }
                __syncwarp();
                if (j == n_chunks) break;
            }
            if (!wait_k_warp<kDiag>(mi, B_E16_B, j)) return;
            if (!wait_k_warp<kDiag>(mi, B_AQ_FULL0 + (j & 1), j >> 1)) return;
            tc_fence_after();
            const uint32_t a_re = dlo + ((OFF_AQ + (j & 1) * 2 * kTile) >> 4);
            issue_complex<2, false, false, 2>(acc + 64, acc + 192, x_re, x_re + 32, a_re, a_re + kIm, dhi, I64, 2);
            if (elect_one()) mma_commit(&bars[B_UPD_DONE]);
        }
    } else {
        // Per chunk g, in the order in which the events normally happen: v of chunk g once v of chunk g-1 has been
        // consumed (R of that chunk is built); then the two Gram halves of chunk g, each once its operands are
        // written and the Gram columns have been read out.  Blocking waits: a polling loop here would take issue
        // slots from the warps that do the work.
#pragma unroll 1
        for (int g = 0; g < n_chunks; ++g) {
            if (g > 0 && !wait_k_warp<kDiag>(mi, B_R16_B, g - 1)) return;
            {
                const ChunkInfo cv = ring_get(mi, g);
                if (elect_one()) {
                    mbar_expect_tx(&bars[B_V_FULL], 16384);
                    tma_load_4d(smem + OFF_V, tm_v, &bars[B_V_FULL], 0, cv.h, cv.jg * C, cv.b);
                }
                __syncwarp();
            }
            const int s = g & 1;
            const uint32_t w_re = dlo + ((OFF_WQ + s * 4 * kTile) >> 4), k_re = dlo + ((OFF_KC + s * 2 * kTile) >> 4);
            if (!wait_k_warp<kDiag>(mi, B_PREP_FULL0 + s, g >> 1)) return;
#pragma unroll 1
            for (int gh = 0; gh < 2; ++gh) {
                if (2 * g + gh > 0 && !wait_k_warp<kDiag>(mi, B_GRAM_DRAINED, 2 * g + gh - 1)) return;
                tc_fence_after();
                // rows = [W ; Qt], columns = tokens i.  Re: W_re Kc_re + W_im Kc_im; Im: W_re Kc_im - W_im Kc_re
                if (elect_one()) {
                    const uint32_t d = tmem + TM_GRAM, w_im = w_re + 2 * kIm;
                    const uint32_t k1 = gh ? k_re + kIm : k_re, k2 = gh ? k_re : k_re + kIm;
                    const uint32_t id2 = gh ? I64 | (1u << 14) : I64;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) mma_ss2(d, w_re + 2 * ks, dhi, k1 + 2 * ks, dhi, I64, ks ? 1u : 0u);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) mma_ss2(d, w_im + 2 * ks, dhi, k2 + 2 * ks, dhi, id2, 1u);
                    mma_commit(&bars[B_GRAM_FULL]);
                }
                __syncwarp();
            }
            // PREP has finished chunk g and, before that, described chunk g + 2: time to bring its inputs into L2
            if (g + 2 < n_chunks) {
                const ChunkInfo cp = ring_get(mi, g + 2);
                if (elect_one()) prefetch_chunk(maps, cp);
                __syncwarp();
            }
        }
    }
}

// ---- PREP ---------------------------------------------------------------------------------------------
// e^{-i phi} from the integer phase: the top 23 bits of the turn count make a float in [1, 2); centred to
// [-0.5, 0.5) turns it is well inside the accurate range of the fast sine / cosine.
__device__ __forceinline__ void turns_sincos(uint32_t turns, float *sn, float *cs)
{
    float f = __uint_as_float(0x3f800000u | (turns >> 9)) - 1.0f;
    f -= f >= 0.5f ? 1.0f : 0.0f;
    __sincosf(f * 6.283185307f, sn, cs);
}

// Phase in 2^-32 turns from fp32 arithmetic (one multiply, one conversion).  Inside this kernel the phase only
// feeds sines and cosines of bf16 operands, so the product's fp32 rounding (2^-24 of the angle) is far below what
// matters; the exact double-precision conversion is kept where phases are exported.
__device__ __forceinline__ uint32_t turns_f32(float theta)
{
    return (uint32_t)(unsigned long long)__float2ll_rn(theta * 683565275.6f);
}

// Stable parameterisation (Section 3, Eqs. "param-alpha", "param-theta", "param-beta") from raw fp32 bits, five
// instructions each: sigmoid(x) = 1 / (1 + 2^(-x log2 e)), tanh(x) = 1 - 2 / (1 + 2^(2 x log2 e)), with the
// approximate (2 ulp) exponential and reciprocal of the special-function unit in their flush-to-zero forms, which
// are single instructions.  Both saturate correctly: the exponential overflows to infinity, whose reciprocal is
// zero, or flushes to zero.
__device__ __forceinline__ float rcp1p_ex2(float y)   // 1 / (1 + 2^y)
{
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(y));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
    return r;
}
__device__ __forceinline__ float alpha_from_raw(const Params &p, uint32_t bits)
{
    return fmaf(p.a_range, rcp1p_ex2(__uint_as_float(bits) * -1.4426950408889634f), p.a_lo);
}
__device__ __forceinline__ float theta_from_raw(const Params &p, uint32_t bits)
{
    return fmaf(p.th_m2, rcp1p_ex2(__uint_as_float(bits) * 2.8853900817779268f), p.th_max);
}

// kFused: alpha, theta and beta arrive raw and go through the stable parameterisation here, on the way into the
// operands.  The key is NOT normalised here: with s_t = 1 / (|k_raw,t| + eps), the recurrence on k = s k_raw is the
// recurrence on k_raw itself with beta s^2 in place of beta and v / s in place of v, so the operands carry the raw
// key and the scales enter where beta and v do (SOLVE and CHAIN); |k_raw,t|^2 is the diagonal of the chunk's Gram
// matrix, which the tensor core computes anyway.
template <bool kFused, bool kDiag>
__device__ __forceinline__ void run_prep(uint8_t *smem, Misc &mi, uint32_t tmem, const Maps &maps, const Params &p,
                                         int n_chunks, int pt)
{
    const int jp = pt & 31, tq = pt >> 5;   // channel pair (channels 2jp, 2jp+1), token octet (8 tokens)
    bool dead = false;
    // this role also reads the finished outputs out of tensor memory (its warps cover the four lane quadrants
    // twice: the first four take rho's real part, the others the imaginary part)
    const int lane = pt & 31, quad = (pt >> 5) & 3, half = pt >> 7;
    const int c = quad * 32 + lane;
    const uint32_t tlane = tmem + ((uint32_t)(quad * 32) << 16);
    auto drain_outputs = [&](int jd) {           // rho of chunk jd -> bf16 staging tiles [t][128]
        if (!dead && !wait_k<kDiag>(mi, B_UPD_DONE, jd)) dead = true;
        // the Re staging tile is shared by all chunks: the store of chunk jd-1 must have read it
        if (jd >= 1 && !dead && !wait_k<kDiag>(mi, B_STORE_DONE0 + ((jd - 1) & 1), (jd - 1) >> 1)) dead = true;
        tc_fence_after();
        if (half == 0 || p.has_o_im) {
            // Tensor memory is read in the 16-lane x 256-bit fragment shape (thread T: channel rows T / 4 and T / 4 + 8,
            // token pairs 2 (T % 4) of every block of eight tokens), whose bf16 pairs are exactly the fragments of a
            // transposing 8 x 8 matrix store: four matrices (one block of eight tokens x four groups of eight
            // channels) per instruction instead of one 2-byte store per value.  The staging tiles hold 64 channels
            // per 128-byte row in the copy engine's 128-byte swizzle, so the 32 row pieces of one store fall into
            // different banks.
            const uint32_t flip = half ? 0x80008000u : 0u;   // o = conj(rho)
            const int r8 = lane & 7, chunk = (quad & 1) * 4 + (lane >> 3);
            uint32_t st = smem_u32(smem + (half ? OFF_AQ + (jd & 1) * 2 * kTile : OFF_OST)) + (quad >> 1) * kTile +
                          (uint32_t)(r8 * 128 + ((chunk ^ r8) << 4));
            uint32_t ta = tlane + TM_ACC + 64 + 128 * half;
#pragma unroll 1
            for (int ch = 0; ch < 2; ++ch, st += 4 * 1024, ta += 32) {
                uint32_t ra[16], rb[16];
                tmem_ld_16x256b_x4(ta, ra);
                tmem_ld_16x256b_x4(ta + (16u << 16), rb);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    stmatrix_x4_trans(st + i * 1024,
                                      pack_bf16(__uint_as_float(ra[4 * i]), __uint_as_float(ra[4 * i + 1])) ^ flip,
                                      pack_bf16(__uint_as_float(ra[4 * i + 2]), __uint_as_float(ra[4 * i + 3])) ^ flip,
                                      pack_bf16(__uint_as_float(rb[4 * i]), __uint_as_float(rb[4 * i + 1])) ^ flip,
                                      pack_bf16(__uint_as_float(rb[4 * i + 2]), __uint_as_float(rb[4 * i + 3])) ^ flip);
                }
            }
        }
        fence_async_smem();
        tc_fence_before();
        warp_arrive(&mi.bars[B_O_STAGED]);
    };
    ChunkCursor cur = ChunkCursor::load(mi.cursor_raw);   // at chunk 2: chunks 0 and 1 were published before the roles started
#pragma unroll 1
    for (int j = 0; j < n_chunks + 2; ++j) {
        const bool live = j < n_chunks;          // after the last chunk only the outputs of two chunks are left
        const int s = j & 1, ring = j & 3;
        float base0 = 1.f, base1 = 1.f, ainv0 = 1.f, ainv1 = 1.f;
        float2 g0 = make_float2(1.f, 0.f), g1 = g0;   // gamma_t = a_t e^{i phi_t} of the two coordinates
        uint32_t tb0 = 0u, tb1 = 0u;
        size_t off = 0, step = 0;                // byte offset of this thread's first token in q/k/alpha/theta
        int nt = 0;                              // real tokens in this thread's octet
        // Inputs of token i of the octet, alpha and theta as raw bits.  Beyond the end of the sequence nothing is
        // loaded and the registers keep what they held (neutral values at first, then an earlier token's): such
        // tokens have beta = 0 and stored-nowhere outputs, so any finite operand rows do for them; the chunk's
        // closing factor comes from pass 1, which does count them as neutral.
        struct Tok { uint2 al, th, k, q; } tk[kTB];
        auto load_token = [&](Tok &t, int i) {
            const size_t o = off + (size_t)i * step;
            const bool on = i < nt;
            ldg64_if(t.al.x, t.al.y, reinterpret_cast<const char *>(p.alpha) + o, on);
            ldg64_if(t.th.x, t.th.y, reinterpret_cast<const char *>(p.theta) + o, on);
            ldg64_if(t.k.x, t.k.y, reinterpret_cast<const char *>(p.k) + o, on);
            ldg64_if(t.q.x, t.q.y, reinterpret_cast<const char *>(p.q) + o, on);
        };
#pragma unroll
        for (int ii = 0; ii < kTB; ++ii) {
            tk[ii].al = make_uint2(0x3f800000u, 0x3f800000u); tk[ii].th = make_uint2(0u, 0u);
            tk[ii].k = make_uint2(0u, 0u); tk[ii].q = make_uint2(0u, 0u);
        }
        if (live) {
            // chunk j + 2: its description for the other roles (the warp that issues the Gram products reads it once this
            // chunk's tiles are announced, and asks for that chunk's q, k, alpha, theta tiles to be brought into L2)
            if (tq == 0 && j + 2 < n_chunks) {       // (the first warp alone walks the cursor)
                if (pt == 0) ring_put(mi, j + 2, cur.ci);
                cur.next(p);
            }
            const ChunkInfo ci = ring_get(mi, j);
            const int t0 = ci.jg * C, len = min(C, p.T - t0);
            const size_t row0 = ((size_t)ci.b * p.T + t0) * p.H + ci.h;   // token t of this head: row0 + t * H
            nt = min(8, max(0, len - tq * 8));
            // all four arrays have 256 bytes per (token, head): the same byte offset serves them all
            step = (size_t)p.H * 256;
            off = (row0 + (size_t)(tq * 8) * p.H) * 256 + 8 * jp;

            // pass 1: this thread's product of alpha (fp32 products of at most 64 factors: relative error far
            // below bf16's) and sum of the integer phase over its 8 tokens
            uint2 al[8], th[8];                  // raw bits; neutral (alpha = 1, theta = 0) beyond the sequence
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                al[i] = make_uint2(0x3f800000u, 0x3f800000u);
                th[i] = make_uint2(0u, 0u);
                ldg64_if(al[i].x, al[i].y, reinterpret_cast<const char *>(p.alpha) + off + i * step, i < nt);
                ldg64_if(th[i].x, th[i].y, reinterpret_cast<const char *>(p.theta) + off + i * step, i < nt);
            }
            // beta of token pt: fetched now, written after the pass below so that its latency is covered
            float beta_t = 0.f;
            if (pt < len) beta_t = __ldg(p.beta + row0 + (size_t)pt * p.H);
            if (kFused && pt < len) beta_t = rcp1p_ex2(beta_t * -1.4426950408889634f);
            {
                float a0 = 1.f, a1 = 1.f;
                uint32_t u0 = 0u, u1 = 0u;
                float rs0 = 0.f, rs1 = 0.f;      // fused: sum of 1 / (1 + e^{2b}) over the octet's real tokens
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (kFused) {   // beyond the sequence the defaults are not raw values: skipped, i.e. neutral
                        if (i < nt) {
                            a0 *= fmaxf(alpha_from_raw(p, al[i].x), 9.0e-14f);
                            a1 *= fmaxf(alpha_from_raw(p, al[i].y), 9.0e-14f);
                            rs0 += rcp1p_ex2(__uint_as_float(th[i].x) * 2.8853900817779268f);
                            rs1 += rcp1p_ex2(__uint_as_float(th[i].y) * 2.8853900817779268f);
                        }
                        continue;
                    }
                    a0 *= fmaxf(__uint_as_float(al[i].x), 9.0e-14f);           // floor e^-30, as in log_decay
                    a1 *= fmaxf(__uint_as_float(al[i].y), 9.0e-14f);
                    u0 += turns_f32(__uint_as_float(th[i].x));
                    u1 += turns_f32(__uint_as_float(th[i].y));
                }
                if (kFused) {   // sum of theta_max tanh(b) = theta_max (n - 2 sum r): at most 8 theta_max, one rounding
                    u0 = turns_f32(fmaf(p.th_m2, rs0, p.th_max * (float)nt));
                    u1 = turns_f32(fmaf(p.th_m2, rs1, p.th_max * (float)nt));
                }
                *reinterpret_cast<float2 *>(&mi.part_lg[s][tq][2 * jp]) = make_float2(a0, a1);
                *reinterpret_cast<uint2 *>(&mi.part_turns[s][tq][2 * jp]) = make_uint2(u0, u1);
            }
            if (pt < C) mi.beta[ring][pt] = beta_t;
#pragma unroll
            for (int ii = 0; ii < kTB; ++ii) load_token(tk[ii], ii);
            // The only barrier of the role.  The partial sums are kept two chunks deep: a warp that runs ahead
            // writes the other copy, and cannot come back to this one before everybody has passed the next barrier.
            if (role_sync_or(2, kPrepThreads, dead || mi.abort)) break;
            // octet tq starts from the product of the octets before it; octet 0 instead multiplies all eight:
            // the chunk totals a_C e^{i phi_C}, applied by the next state pass
            const int n_before = tq == 0 ? 8 : tq;
#pragma unroll 1
            for (int gq = 0; gq < n_before; ++gq) {
                const float2 pl = *reinterpret_cast<const float2 *>(&mi.part_lg[s][gq][2 * jp]);
                const uint2 pu = *reinterpret_cast<const uint2 *>(&mi.part_turns[s][gq][2 * jp]);
                base0 *= pl.x; base1 *= pl.y; tb0 += pu.x; tb1 += pu.y;
            }
            {   // gamma at the start of the group (group 0: of the whole chunk, for the next state pass)
                float cs, sn;
                turns_sincos(tb0, &sn, &cs);
                g0 = make_float2(base0 * cs, base0 * sn);
                turns_sincos(tb1, &sn, &cs);
                g1 = make_float2(base1 * cs, base1 * sn);
                if (tq == 0) {
                    // the integer phase the chunk closes with: what the operands' angles are derived from, exported
                    // on request so that it can be compared bit for bit
                    if (!kFused && p.phase_out)
                        *reinterpret_cast<uint2 *>(p.phase_out + ((size_t)ci.bh * p.NC + ci.jg) * M + 2 * jp) = make_uint2(tb0, tb1);
                    *reinterpret_cast<float2 *>(&mi.close_re[ring][2 * jp]) = make_float2(g0.x, g1.x);
                    *reinterpret_cast<float2 *>(&mi.close_im[ring][2 * jp]) = make_float2(g0.y, g1.y);
                    g0 = make_float2(1.f, 0.f); g1 = g0; base0 = 1.f; base1 = 1.f;
                }
                ainv0 = fminf(__fdividef(1.0f, base0), 5.5e34f);          // 1/a, capped at e^80
                ainv1 = fminf(__fdividef(1.0f, base1), 5.5e34f);
            }

            // (the slot's tiles, last read by the state update of chunk j-2, are free once that chunk's products are
            // complete, which the read-out of its outputs below waits for)
        }
        // the state update of chunk j-2 has just finished (it freed Kc above): read out that chunk's outputs,
        // so that rho is free when the next chunk's first product is issued
        if (j >= 2) drain_outputs(j - 2);
        if (!live) continue;

        // pass 2: rotated / decayed operands.  A rolled loop over groups of kTB tokens keeps the code small; each
        // token's inputs (from L1 / L2: pass 1 or the prefetch warp brought them in) are fetched into the
        // registers of the token kTB places before it as soon as that one has been worked on.
        const uint32_t wq_re = smem_u32(smem) + OFF_WQ + s * 4 * kTile + tq * 1024 + (jp & 3) * 4;   // + row, swizzle
        const uint32_t kc_re = smem_u32(smem) + OFF_KC + s * 2 * kTile + tq * 1024 + (jp & 3) * 4;
        // The thread's two coordinates go through the arithmetic side by side as packed pairs (one instruction for both):
        // this role is short of issue slots, not of floating-point throughput.
        float2 gx2 = make_float2(g0.x, g1.x), gy2 = make_float2(g0.y, g1.y), ainv2 = make_float2(ainv0, ainv1);
#pragma unroll 1
        for (int h = 0; h < 8 / kTB; ++h) {
#pragma unroll
            for (int ii = 0; ii < kTB; ++ii) {
                const int i = h * kTB + ii;
                // gamma_t = gamma_{t-1} alpha_t e^{i theta_t}; 1/a_t alongside (capped at e^80)
                const float2 al2 = make_float2(
                    fmaxf(kFused ? alpha_from_raw(p, tk[ii].al.x) : __uint_as_float(tk[ii].al.x), 9.0e-14f),   // floor e^-30
                    fmaxf(kFused ? alpha_from_raw(p, tk[ii].al.y) : __uint_as_float(tk[ii].al.y), 9.0e-14f));
                float2 cs2, sn2;
                __sincosf(kFused ? theta_from_raw(p, tk[ii].th.x) : __uint_as_float(tk[ii].th.x), &sn2.x, &cs2.x);
                __sincosf(kFused ? theta_from_raw(p, tk[ii].th.y) : __uint_as_float(tk[ii].th.y), &sn2.y, &cs2.y);
                const float2 lr2 = __fmul2_rn(al2, cs2), li2 = __fmul2_rn(al2, sn2);
                const float2 gxn = __ffma2_rn(gy2, make_float2(-li2.x, -li2.y), __fmul2_rn(gx2, lr2));
                gy2 = __ffma2_rn(gy2, lr2, __fmul2_rn(gx2, li2));
                gx2 = gxn;
                ainv2 = __fmul2_rn(ainv2, make_float2(__fdividef(1.0f, al2.x), __fdividef(1.0f, al2.y)));
                ainv2 = make_float2(fminf(ainv2.x, 5.5e34f), fminf(ainv2.y, 5.5e34f));
                const uint32_t k0 = tk[ii].k.x, k1 = tk[ii].k.y, q0 = tk[ii].q.x, q1 = tk[ii].q.y;
                const float2 kr2 = make_float2(__uint_as_float(k0 << 16), __uint_as_float(k1 << 16));
                const float2 ki2 = make_float2(__uint_as_float(k0 & 0xffff0000u), __uint_as_float(k1 & 0xffff0000u));
                const float2 qr2 = make_float2(__uint_as_float(q0 << 16), __uint_as_float(q1 << 16));
                const float2 qi2 = make_float2(__uint_as_float(q0 & 0xffff0000u), __uint_as_float(q1 & 0xffff0000u));
                const float2 ngy2 = make_float2(-gy2.x, -gy2.y);
                const float2 wr2 = __ffma2_rn(gy2, ki2, __fmul2_rn(gx2, kr2));     // W = conj(gamma) k
                const float2 wi2 = __ffma2_rn(ngy2, kr2, __fmul2_rn(gx2, ki2));
                const float2 tr2 = __ffma2_rn(gy2, qi2, __fmul2_rn(gx2, qr2));     // Qt = conj(gamma) q
                const float2 ti2 = __ffma2_rn(ngy2, qr2, __fmul2_rn(gx2, qi2));
                const float2 cr2 = __fmul2_rn(__fmul2_rn(wr2, ainv2), ainv2);      // Kc = k / gamma = W / a^2
                const float2 ci2 = __fmul2_rn(__fmul2_rn(wi2, ainv2), ainv2);
                load_token(tk[ii], i + kTB);
                const int o1 = i * 128 + ((((jp >> 2) ^ i) & 7) << 4);      // row i of the octet's 8-row swizzle atom
                sts32(wq_re + o1, pack_bf16(wr2.x, wr2.y));
                sts32(wq_re + 2 * kTile + o1, pack_bf16(wi2.x, wi2.y));
                sts32(wq_re + kTile + o1, pack_bf16(tr2.x, tr2.y));
                sts32(wq_re + 3 * kTile + o1, pack_bf16(ti2.x, ti2.y));
                sts32(kc_re + o1, pack_bf16(cr2.x, cr2.y));
                sts32(kc_re + kTile + o1, pack_bf16(ci2.x, ci2.y));
            }
        }
        fence_async_smem();
        warp_arrive(&mi.bars[B_PREP_FULL0 + s]);
    }
}

// ---- SOLVE --------------------------------------------------------------------------------------------
// NRT stacked 16 x 8 tiles of a complex product A B, operands in the solve scratch (fp32, row stride LS, Re at
// shared address `lx`, Im 64 rows further): tile rt covers rows a_row0 + 16 rt .. + 15 of A and k-steps
// s0 <= s < s1[rt] (8 columns of A / rows of B per step; s1[0] <= s1[1]).  B's 8 columns start at b_col0.  Each
// tile keeps four independent accumulators (Re: ar br and -ai bi; Im: ar bi and ai br), summed at the end, so
// that consecutive tensor-core instructions do not wait for one another.
template <int NRT>
__device__ __forceinline__ void cmma_tiles(float (&cr)[NRT][4], float (&ci)[NRT][4], uint32_t lx, int a_row0, int a_col0,
                                           int b_row0, int b_col0, int s0, int s1a, int s1b, int lane)
{
    constexpr uint32_t kIm = 64 * LS * 4;
    const int g = lane >> 2, tg = lane & 3, m = lane >> 3, r = lane & 7;
    float acc[NRT][4][4];
#pragma unroll
    for (int rt = 0; rt < NRT; ++rt)
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) acc[rt][x][y] = 0.f;
    // lane's row address for the A blocks: block m = (rows 0-7 | 8-15) x (k 0-3 | 4-7)
    uint32_t a_addr = lx + (uint32_t)(((a_row0 + r + 8 * (m & 1)) * LS + a_col0 + 8 * s0 + 4 * (m >> 1)) * 4);
    uint32_t b_addr = lx + (uint32_t)(((b_row0 + 8 * s0 + tg) * LS + b_col0 + g) * 4);
#pragma unroll 4
    for (int s = s0; s < s1b; ++s, a_addr += 32, b_addr += 8 * LS * 4) {
        uint32_t br[2], bi[2], nbi[2];
        br[0] = lds32(b_addr);
        br[1] = lds32(b_addr + 4 * LS * 4);
        bi[0] = lds32(b_addr + kIm);
        bi[1] = lds32(b_addr + kIm + 4 * LS * 4);
        nbi[0] = bi[0] ^ 0x80000000u;
        nbi[1] = bi[1] ^ 0x80000000u;
#pragma unroll
        for (int rt = 0; rt < NRT; ++rt) {
            if (NRT == 2 && rt == 0 && s >= s1a) continue;
            uint32_t ar[4], ai[4];
            ldmatrix_x4(ar, a_addr + rt * 16 * LS * 4);
            ldmatrix_x4(ai, a_addr + rt * 16 * LS * 4 + kIm);
            mma_tf32(acc[rt][0], ar, br);
            mma_tf32(acc[rt][1], ai, nbi);
            mma_tf32(acc[rt][2], ar, bi);
            mma_tf32(acc[rt][3], ai, br);
        }
    }
#pragma unroll
    for (int rt = 0; rt < NRT; ++rt)
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            cr[rt][y] = acc[rt][0][y] + acc[rt][1][y];
            ci[rt][y] = acc[rt][2][y] + acc[rt][3][y];
        }
}
// Store a 16 x 8 accumulator tile (times `scale`) at rows row0.., columns col0.. of the scratch.
__device__ __forceinline__ void store_tile_s(const float (&cr)[4], const float (&ci)[4], float scale, uint32_t lx, int row0,
                                             int col0, int lane)
{
    constexpr uint32_t kIm = 64 * LS * 4;
    const int g = lane >> 2, tg = lane & 3;
    const uint32_t o = lx + (uint32_t)(((row0 + g) * LS + col0 + 2 * tg) * 4);
    sts64(o, __float_as_uint(scale * cr[0]), __float_as_uint(scale * cr[1]));
    sts64(o + 8 * LS * 4, __float_as_uint(scale * cr[2]), __float_as_uint(scale * cr[3]));
    sts64(o + kIm, __float_as_uint(scale * ci[0]), __float_as_uint(scale * ci[1]));
    sts64(o + kIm + 8 * LS * 4, __float_as_uint(scale * ci[2]), __float_as_uint(scale * ci[3]));
}

// kFused: the diagonal of the Gram matrix is |k_raw,t|^2 (conj(W) Kc = |k|^2 whatever gamma is); the thread that
// drains Kt row t turns it into s_t = 1 / (|k_raw,t| + eps), scales its row of L by beta_t s_t^2, and leaves
// beta_t s_t (the column scale of the M operand, which then maps the normalised R to E / s) and -s_t (for CHAIN's
// R = v - s W_raw^* S_0) in shared memory.
template <bool kFused, bool kDiag>
__device__ __forceinline__ void run_solve(uint8_t *smem, Misc &mi, uint32_t tmem, const Params &p, int n_chunks, int st)
{
    const int lane = st & 31, w = st >> 5;    // w = TMEM lane quadrant of this warp
    constexpr uint32_t kIm = 64 * LS * 4;     // Re -> Im in the scratch
    const uint32_t sbase = smem_u32(smem), lx = sbase + OFF_LX;
    const uint32_t tlane = tmem + ((uint32_t)(w * 32) << 16);
    const int row = w * 32 + lane;            // Gram row held by this thread: < 64 -> Kt row, else Aq row
    bool dead = false;
#pragma unroll 1
    for (int j = 0; j < n_chunks; ++j) {
        if (role_sync_or(1, kSolveThreads, dead || mi.abort)) break;   // also: scratch of the last chunk is free
        const int s = j & 1, ring = j & 3;
        // The Aq tile of this slot also staged o_im of chunk j-2: its rows are written straight from the drain,
        // so the warps that hold them wait for that store first.
        if (row >= 64 && j >= 2 && !dead && !wait_k<kDiag>(mi, B_STORE_DONE0 + s, (j >> 1) - 1)) dead = true;
        // ---- drain the two Gram halves (Re, then Im), 32 columns at a time
        float bt = 0.f;                           // beta of this thread's Kt row (PREP wrote it before the Gram ran)
#pragma unroll 1
        for (int im = 0; im < 2; ++im) {
            if (!dead && !wait_k<kDiag>(mi, B_GRAM_FULL, 2 * j + im)) dead = true;
            tc_fence_after();
            if (im == 0 && row < 64) bt = mi.beta[ring][row];
#pragma unroll 1
            for (int it = 0; it < 2; ++it) {
                // fused: the piece that holds this warp's diagonal entries of Re Kt comes first
                const bool diag = kFused && im == 0 && it == 0 && row < 64;
                const int hc = (kFused && im == 0 && w == 1) ? 1 - it : it;
                uint32_t r[32];
                tmem_ld<32>(tlane + TM_GRAM + 32 * hc, r);
                tc_wait_ld();
                if (it == 1) {
                    tc_fence_before();
                    warp_arrive(&mi.bars[B_GRAM_DRAINED]);
                }
                if (diag) {                        // r[lane] by a select tree on the lane's bits
                    uint32_t d[16];
#pragma unroll
                    for (int x = 0; x < 16; ++x) d[x] = (lane & 16) ? r[16 + x] : r[x];
#pragma unroll
                    for (int x = 0; x < 8; ++x) d[x] = (lane & 8) ? d[8 + x] : d[x];
#pragma unroll
                    for (int x = 0; x < 4; ++x) d[x] = (lane & 4) ? d[4 + x] : d[x];
#pragma unroll
                    for (int x = 0; x < 2; ++x) d[x] = (lane & 2) ? d[2 + x] : d[x];
                    float n = fmaxf(__uint_as_float((lane & 1) ? d[1] : d[0]), 0.f), sc;
                    asm("sqrt.approx.ftz.f32 %0, %0;" : "+f"(n));
                    // (|k_raw| + eps below 1e-18 counts as 1e-18: s^2 stays finite, and a zero key stays a zero key)
                    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(sc) : "f"(fmaxf(n + p.eps, 1.0e-18f)));
                    mi.kscale[ring][row] = sc;
                    mi.beta[ring][row] = bt * sc;
                    bt = bt * sc * sc;
                    warp_arrive(&mi.bars[B_NORM_FULL]);
                }
                if (row < 64) {                   // L = D_beta Kt, strictly lower
                    const uint32_t dst = lx + im * kIm + (uint32_t)((row * LS + 32 * hc) * 4);
                    // no mask: the substitution reads only entries below the diagonal of an 8x8 block and then
                    // overwrites the whole block; the merges read whole blocks strictly below the diagonal
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        const float2 bt2 = make_float2(bt, bt);
                        const float2 lo = __fmul2_rn(bt2, make_float2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])));
                        const float2 hi = __fmul2_rn(bt2, make_float2(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3])));
                        sts128(dst + 4 * i, __float_as_uint(lo.x), __float_as_uint(lo.y), __float_as_uint(hi.x), __float_as_uint(hi.y));
                    }
                } else {                          // Aq, lower incl. diagonal, as a bf16 operand tile
                    const int t = row - 64;
                    const uint32_t tile = sbase + OFF_AQ + (s * 2 + im) * kTile;
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) {
                        uint32_t wv[4];
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            const int ii = 32 * hc + 8 * c8 + 2 * x;
                            wv[x] = pack_bf16(ii <= t ? __uint_as_float(r[8 * c8 + 2 * x]) : 0.f,
                                              ii + 1 <= t ? __uint_as_float(r[8 * c8 + 2 * x + 1]) : 0.f);
                        }
                        sts128(tile + sw_off(t, 32 * hc + 8 * c8), wv[0], wv[1], wv[2], wv[3]);
                    }
                }
            }
        }
        fence_async_smem();
        warp_arrive(&mi.bars[B_AQ_FULL0 + s]);
        role_sync(1, kSolveThreads);

        // ---- X = (I + L)^{-1} in place.  Diagonal 8x8 blocks: lane = column c of block blk solves
        // (I + L) x = e_c right-looking (after x_i is final every later row is updated at once).
        if (w < 2) {
            const int o = 8 * (4 * w + (lane >> 3)), c = lane & 7;
            const uint32_t blk = lx + (uint32_t)((o * LS + o) * 4);
            float xr[8], xi[8];
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                xr[r] = r == c ? 1.f : 0.f;
                xi[r] = 0.f;
            }
#pragma unroll
            for (int i = 0; i < 7; ++i) {
                const float vr = xr[i], vi = xi[i];      // zero above the diagonal (i < c)
#pragma unroll
                for (int r = i + 1; r < 8; ++r) {
                    const float lr_ = __uint_as_float(lds32(blk + (r * LS + i) * 4));
                    const float li_ = __uint_as_float(lds32(blk + kIm + (r * LS + i) * 4));
                    xr[r] -= lr_ * vr - li_ * vi;
                    xi[r] -= lr_ * vi + li_ * vr;
                }
            }
            __syncwarp();                     // every lane has read its L block before it is overwritten
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                sts32(blk + (r * LS + c) * 4, __float_as_uint(xr[r]));
                sts32(blk + kIm + (r * LS + c) * 4, __float_as_uint(xi[r]));
            }
        }
        role_sync(1, kSolveThreads);
        // ---- three merge levels: X[lower-left] = -X[lower-right] (L[lower-left] X[upper-left]); the intermediate
        // product T is parked in the (unused) block above the diagonal
        {   // level 0: 8 -> 16.  Warp w merges 16-block w.  The m16 tile is placed on the whole 16-row block, so
            // its lower eight rows (fragment elements 2, 3) are the rows that matter.
            const int o = 16 * w;
            const int g = lane >> 2, tg = lane & 3;
            float cr[1][4], ci[1][4];
            cmma_tiles<1>(cr, ci, lx, o, o, o, o, 0, 1, 1, lane);               // rows 8..15: L21 X11
            const uint32_t tpos = lx + (uint32_t)(((o + g) * LS + o + 8 + 2 * tg) * 4);   // rows o.., columns o+8..
            sts64(tpos, __float_as_uint(cr[0][2]), __float_as_uint(cr[0][3]));
            sts64(tpos + kIm, __float_as_uint(ci[0][2]), __float_as_uint(ci[0][3]));
            __syncwarp();
            cmma_tiles<1>(cr, ci, lx, o, o + 8, o, o + 8, 0, 1, 1, lane);       // rows 8..15: X22 T
            const uint32_t xpos = lx + (uint32_t)(((o + 8 + g) * LS + o + 2 * tg) * 4);
            sts64(xpos, __float_as_uint(-cr[0][2]), __float_as_uint(-cr[0][3]));
            sts64(xpos + kIm, __float_as_uint(-ci[0][2]), __float_as_uint(-ci[0][3]));
            // the block above the diagonal held T; later levels read the whole 16x16 diagonal block
            __syncwarp();
            sts64(tpos, 0u, 0u);
            sts64(tpos + kIm, 0u, 0u);
        }
        role_sync(1, kSolveThreads);
        {   // level 1: 16 -> 32.  Warp pair pr merges 32-block pr; warp's column tile nt of the 16 columns
            const int pr = w >> 1, nt = w & 1;
            const int r0 = 32 * pr + 16, c0 = 32 * pr;
            float cr[1][4], ci[1][4];
            cmma_tiles<1>(cr, ci, lx, r0, c0, c0, c0 + 8 * nt, nt, 2, 2, lane);
            store_tile_s(cr[0], ci[0], 1.f, lx, c0, r0 + 8 * nt, lane);          // T at block (b0, b1)
            role_sync(1, kSolveThreads);
            cmma_tiles<1>(cr, ci, lx, r0, r0, c0, r0 + 8 * nt, 0, 2, 2, lane);
            store_tile_s(cr[0], ci[0], -1.f, lx, r0, c0 + 8 * nt, lane);
        }
        role_sync(1, kSolveThreads);
        {   // level 2: 32 -> 64.  T in the top-right quadrant; warp w owns column tile w of the 32 columns
            const int nt = w;
            float cr[2][4], ci[2][4];
            cmma_tiles<2>(cr, ci, lx, 32, 0, 0, 8 * nt, nt, 4, 4, lane);
            store_tile_s(cr[0], ci[0], 1.f, lx, 0, 32 + 8 * nt, lane);
            store_tile_s(cr[1], ci[1], 1.f, lx, 16, 32 + 8 * nt, lane);
            role_sync(1, kSolveThreads);
            cmma_tiles<2>(cr, ci, lx, 32, 32, 0, 32 + 8 * nt, 0, 2, 4, lane);    // X22 lower triangular
            store_tile_s(cr[0], ci[0], -1.f, lx, 32, 8 * nt, lane);
            store_tile_s(cr[1], ci[1], -1.f, lx, 48, 8 * nt, lane);
        }
        role_sync(1, kSolveThreads);

        // ---- M_beta = X D_beta as a bf16 operand tile, once E of the previous chunk has read the old one
        if (j >= 1 && !dead && !wait_k<kDiag>(mi, B_E_DONE, j - 1)) dead = true;
        {
            const int t = st >> 1, part = st & 1;   // row t, columns 32 part .. 32 part + 31
            const uint32_t src = lx + (uint32_t)((t * LS + 32 * part) * 4);
            const uint32_t bsrc = smem_u32(&mi.beta[ring][32 * part]);
#pragma unroll 1
            for (int cidx = 0; cidx < 4; ++cidx) {
                uint32_t wr[4], wi[4];
#pragma unroll
                for (int hx = 0; hx < 2; ++hx) {
                    const uint4 b4 = lds128(bsrc + (8 * cidx + 4 * hx) * 4);
                    const uint4 r4 = lds128(src + (8 * cidx + 4 * hx) * 4);
                    const uint4 i4 = lds128(src + kIm + (8 * cidx + 4 * hx) * 4);
                    const int i0 = 32 * part + 8 * cidx + 4 * hx;
                    const float m0 = i0 <= t ? __uint_as_float(b4.x) : 0.f, m1 = i0 + 1 <= t ? __uint_as_float(b4.y) : 0.f;
                    const float m2 = i0 + 2 <= t ? __uint_as_float(b4.z) : 0.f, m3 = i0 + 3 <= t ? __uint_as_float(b4.w) : 0.f;
                    wr[2 * hx] = pack_bf16(__uint_as_float(r4.x) * m0, __uint_as_float(r4.y) * m1);
                    wr[2 * hx + 1] = pack_bf16(__uint_as_float(r4.z) * m2, __uint_as_float(r4.w) * m3);
                    wi[2 * hx] = pack_bf16(__uint_as_float(i4.x) * m0, __uint_as_float(i4.y) * m1);
                    wi[2 * hx + 1] = pack_bf16(__uint_as_float(i4.z) * m2, __uint_as_float(i4.w) * m3);
                }
                const uint32_t off = sbase + OFF_MB + sw_off(t, 32 * part + 8 * cidx);
                sts128(off, wr[0], wr[1], wr[2], wr[3]);
                sts128(off + kTile, wi[0], wi[1], wi[2], wi[3]);
            }
        }
        fence_async_smem();
        warp_arrive(&mi.bars[B_MB_FULL]);
    }
}

// ---- CHAIN --------------------------------------------------------------------------------------------
template <bool kFused, bool kDiag>
__device__ __forceinline__ void run_chain(uint8_t *smem, Misc &mi, uint32_t tmem, const Params &p, int n_chunks, int ct)
{
    const int lane = ct & 31, warp = ct >> 5;
    const int quad = warp & 3, half = warp >> 2;
    const int c = quad * 32 + lane;            // value channel = TMEM lane
    const int j0 = half * 32;                  // this warp's complex rows in the state pass
    const uint32_t tlane = tmem + ((uint32_t)(quad * 32) << 16);
    const uint32_t sv = smem_u32(smem) + OFF_V + 2 * c;   // v[t][c], rows of 256 bytes

    ChunkInfo prev_ci = ring_get(mi, 0);
#pragma unroll 1
    for (int j = 0; j <= n_chunks; ++j) {
        // ---- state pass: S_0 of this chunk = e^{i phi_C} a_C (accumulated state of the previous chunk)
        if (j > 0) {
            if (!wait_k_warp<kDiag>(mi, B_UPD_DONE, j - 1)) return;
            tc_fence_after();
        }
        const bool fin = j == n_chunks;
        const ChunkInfo ci = fin ? prev_ci : ring_get(mi, j);
        const float *close_re = mi.close_re[(j - 1) & 3], *close_im = mi.close_im[(j - 1) & 3];
        const float *src = nullptr;
        if (fin || ci.first) {
            // A unit ends (chunk j - 1 was its last): its final state e^{i phi_C} a_C S goes to S_T (last time
            // slice) or to the hand-off buffer, where the CTA that runs the next slice is told about it.
            if (j > 0) {
                float *dst = prev_ci.seq_last ? p.S_T : p.handoff;
                if (dst) {
                    dst += (size_t)prev_ci.bh * DK * DV + c;
#pragma unroll 1
                    for (int pc = 0; pc < 4; ++pc) {
                        uint32_t sre[8], sim[8];
                        const int jb = j0 + 8 * pc;
                        tmem_ld8(tlane + TM_S32 + jb, sre);
                        tmem_ld8(tlane + TM_S32 + 64 + jb, sim);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float clx = close_re[jb + i], cly = close_im[jb + i];
                            const float xr = __uint_as_float(sre[i]), xi = __uint_as_float(sim[i]);
                            // (the same roundings as the state pass, so that a state handed over through memory
                            // continues with the very bits an uncut sequence carries on chip)
                            __stcg(dst + (size_t)(2 * (jb + i)) * DV, __fmaf_rn(-cly, xi, __fmul_rn(clx, xr)));
                            __stcg(dst + (size_t)(2 * (jb + i) + 1) * DV, __fmaf_rn(cly, xr, __fmul_rn(clx, xi)));
                        }
                    }
                }
                if (!prev_ci.seq_last) {     // one count per warp: the next piece may start once all eight have arrived
                    __threadfence();
                    __syncwarp();
                    if (lane == 0 && !(kDiag && p.withhold)) atomicAdd(p.flags + prev_ci.bh, 1u);
                }
            }
            if (fin) break;
            if (ci.seq_first) {
                src = p.S0 ? p.S0 + (size_t)ci.bh * DK * DV + c : nullptr;
            } else {
                // the boundary state of this sequence's previous time slice must have been written (eight warp
                // counts per slice); bounded like every other wait, warp-uniform result
                int ok = 1;
                if (lane == 0) {
                    const uint32_t want = ci.want, t0 = (uint32_t)clock();
                    uint32_t seen;
                    do {
                        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(p.flags + ci.bh) : "memory");
                        if (seen >= want) break;
                        __nanosleep(200);
                    } while (!mi.abort && (uint32_t)clock() - t0 < (kDiag ? p.wait_limit : 0x80000000u));
                    ok = seen >= want;
                    if (!ok) mi.abort = 1;
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                __threadfence();
                if (!ok) return;
                src = p.handoff + (size_t)ci.bh * DK * DV + c;
            }
        }
        // 16 complex rows at a time: fp32 state (decayed and rotated in place) and its bf16 copy, the A operand
#pragma unroll 1
        for (int pc = 0; pc < 2; ++pc) {
            uint32_t sre[16], sim[16], pk[8];
            const int jb = j0 + 16 * pc;
            if (ci.first) {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    sre[i] = src ? __float_as_uint(__ldcg(src + (size_t)(2 * (jb + i)) * DV)) : 0u;
                    sim[i] = src ? __float_as_uint(__ldcg(src + (size_t)(2 * (jb + i) + 1) * DV)) : 0u;
                }
            } else {
                tmem_ld<16>(tlane + TM_S32 + jb, sre);
                tmem_ld<16>(tlane + TM_S32 + 64 + jb, sim);
                tc_wait_ld();
                // two rows per instruction (packed pairs): (re, im) <- (c_re re - c_im im, c_re im + c_im re)
                const uint32_t cre = smem_u32(close_re + jb), cim = smem_u32(close_im + jb);
#pragma unroll
                for (int i = 0; i < 16; i += 4) {
                    const uint4 c4 = lds128(cre + 4 * i), d4 = lds128(cim + 4 * i);
#pragma unroll
                    for (int x = 0; x < 4; x += 2) {
                        const float2 cr2 = make_float2(__uint_as_float(x ? c4.z : c4.x), __uint_as_float(x ? c4.w : c4.y));
                        const float2 ci2 = make_float2(__uint_as_float(x ? d4.z : d4.x), __uint_as_float(x ? d4.w : d4.y));
                        const float2 xr2 = make_float2(__uint_as_float(sre[i + x]), __uint_as_float(sre[i + x + 1]));
                        const float2 xi2 = make_float2(__uint_as_float(sim[i + x]), __uint_as_float(sim[i + x + 1]));
                        const float2 nr2 = __ffma2_rn(make_float2(-ci2.x, -ci2.y), xi2, __fmul2_rn(cr2, xr2));
                        const float2 ni2 = __ffma2_rn(ci2, xr2, __fmul2_rn(cr2, xi2));
                        sre[i + x] = __float_as_uint(nr2.x); sre[i + x + 1] = __float_as_uint(nr2.y);
                        sim[i + x] = __float_as_uint(ni2.x); sim[i + x + 1] = __float_as_uint(ni2.y);
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) pk[i] = pack_bf16(__uint_as_float(sre[2 * i]), __uint_as_float(sre[2 * i + 1]));
            tmem_st8(tlane + TM_X16 + jb / 2, pk);
#pragma unroll
            for (int i = 0; i < 8; ++i) pk[i] = pack_bf16(__uint_as_float(sim[2 * i]), __uint_as_float(sim[2 * i + 1]));
            tmem_st8(tlane + TM_X16 + 32 + jb / 2, pk);
            tmem_st<16>(tlane + TM_S32 + jb, sre);
            tmem_st<16>(tlane + TM_S32 + 64 + jb, sim);
            tc_wait_st();
            tc_fence_before();
            warp_arrive(&mi.bars[B_S16_A + pc]);   // this half of the operand is complete
        }
        prev_ci = ci;

        // ---- R = V - D1 (ph 0), then E (ph 1), -> bf16 A operand: 64 fp32 accumulator columns of this warp's half
        // (Re for the first four warps, Im for the others), 16 at a time.  D1 and rho_1, which read S_0 from the
        // same columns, are both done when D1 is.
#pragma unroll 1
        for (int ph = 0; ph < 2; ++ph) {
            if (ph == 0) {
                if (!wait_k_warp<kDiag>(mi, B_D1_DONE, j)) return;
                if (!wait_k_warp<kDiag>(mi, B_V_FULL, j)) return;
            } else {
                if (!wait_k_warp<kDiag>(mi, B_E_DONE, j)) return;
            }
            tc_fence_after();
            // The accumulators hold -D1 (ph 0) or E (ph 1): R_re = V + (-D1)_re, R_im = (-D1)_im, E as it is -- only the
            // four warps of the real half add anything, and only in ph 0.
            const bool sub_v = ph == 0 && half == 0;
            // fused: D1 was formed with the raw key, R = V - s D1: the per-token factor s multiplies -D1
            if (kFused && ph == 0 && !wait_k_warp<kDiag>(mi, B_NORM_FULL, j)) return;
            [[maybe_unused]] const uint32_t scp = smem_u32(&mi.kscale[(j & 3)][0]);
            // The second half of the accumulator is read into registers before the first half of the operand is
            // announced: the product which that announcement releases (E = M_beta R goes out in two halves of its K
            // dimension) starts these very accumulator columns from zero, all 64 of them, so a warp that fetched
            // columns 32..63 only after announcing columns 0..31 could find E's partial sums where D1 was.
            uint32_t r[32];
            tmem_ld<32>(tlane + TM_ACC + 128 * half, r);
            tc_wait_ld();
#pragma unroll 1
            for (int pc = 0; pc < 2; ++pc) {       // 32 columns per tensor-memory round trip
                uint32_t pk[16];
                if (kFused && ph == 0) {
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        const uint4 sc4 = lds128(scp + (32 * pc + 2 * i) * 4);
                        r[2 * i] = __float_as_uint(__uint_as_float(sc4.x) * __uint_as_float(r[2 * i]));
                        r[2 * i + 1] = __float_as_uint(__uint_as_float(sc4.y) * __uint_as_float(r[2 * i + 1]));
                        r[2 * i + 2] = __float_as_uint(__uint_as_float(sc4.z) * __uint_as_float(r[2 * i + 2]));
                        r[2 * i + 3] = __float_as_uint(__uint_as_float(sc4.w) * __uint_as_float(r[2 * i + 3]));
                    }
                }
                if (sub_v) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        pk[i] = pack_bf16(add_bf16_f32(lds16(sv + (32 * pc + 2 * i) * 2 * DV), __uint_as_float(r[2 * i])),
                                          add_bf16_f32(lds16(sv + (32 * pc + 2 * i + 1) * 2 * DV), __uint_as_float(r[2 * i + 1])));
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                }
                if (pc == 0) {
                    tmem_ld<32>(tlane + TM_ACC + 128 * half + 32, r);
                    tc_wait_ld();
                }
                // R replaces S_0 in the operand columns: rho_1, the last reader of S_0, must be done
                if (ph == 0 && pc == 0 && !wait_k_warp<kDiag>(mi, B_O1_DONE, j)) return;
                tmem_st<16>(tlane + TM_X16 + 32 * half + 16 * pc, pk);
                tc_wait_st();
                tc_fence_before();
                warp_arrive(&mi.bars[(ph == 0 ? B_R16_A : B_E16_A) + pc]);   // this half of the operand is complete
            }
        }
    }
}

// ---- the kernel ---------------------------------------------------------------------------------------
template <bool kFused, bool kDiag>
__global__ void __launch_bounds__(kThreads, 1)
sfda_forward_ws_kernel(const __grid_constant__ Maps maps, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Misc &mi = *reinterpret_cast<Misc *>(smem + OFF_MISC);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int n_chunks = ChunkCursor::stream_chunks(p);   // length of this CTA's stream of chunks

    if (tid == 0) {
        auto init = [&](int bar, uint32_t count) { mbar_init(&mi.bars[bar], count); };
        init(B_PREP_FULL0, kPrepWarps); init(B_PREP_FULL1, kPrepWarps);
        init(B_STORE_DONE0, 1); init(B_STORE_DONE1, 1);
        init(B_GRAM_FULL, 1); init(B_GRAM_DRAINED, kSolveWarps);
        init(B_MB_FULL, kSolveWarps); init(B_AQ_FULL0, kSolveWarps); init(B_AQ_FULL1, kSolveWarps);
        init(B_D1_DONE, 2); init(B_O1_DONE, 2); init(B_E_DONE, 2);
        init(B_UPD_DONE, 3);   // the two halves of the state update and rho += Aq E
        init(B_S16_A, kChainWarps); init(B_S16_B, kChainWarps); init(B_R16_A, kChainWarps); init(B_R16_B, kChainWarps);
        init(B_E16_A, kChainWarps); init(B_E16_B, kChainWarps);
        init(B_O_STAGED, kPrepWarps); init(B_V_FULL, 1); init(B_NORM_FULL, 2);
        mi.abort = 0;
        if (kDiag) mi.wait_limit = p.wait_limit;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid == kChainThreads + kSolveThreads) {
        // PREP's first thread walks the stream of chunks for everybody: chunks 0 and 1 are described (and their inputs
        // requested into L2) before the roles start; it goes on from there inside PREP, two chunks ahead
        ChunkCursor cur(p);
#pragma unroll 1
        for (int i = 0; i < 2 && i < n_chunks; ++i) {
            ring_put(mi, i, cur.ci);
            prefetch_chunk(maps, cur.ci);
            cur.next(p);
        }
        cur.store(mi.cursor_raw);
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&mi.tmem_base)));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = mi.tmem_base;

    if (warp < kChainWarps) {
        regs_inc<kRegsWork>();
        run_chain<kFused, kDiag>(smem, mi, tmem, p, n_chunks, tid);
    } else if (warp < kChainWarps + kSolveWarps) {
        regs_inc<kRegsWork>();
        run_solve<kFused, kDiag>(smem, mi, tmem, p, n_chunks, tid - kChainThreads);
    } else if (warp < kChainWarps + kSolveWarps + kPrepWarps) {
        regs_inc<kRegsWork>();
        run_prep<kFused, kDiag>(smem, mi, tmem, maps, p, n_chunks, tid - kChainThreads - kSolveThreads);
    } else {
        regs_dec<kRegsCtrl>();
        const int cw = warp - (kChainWarps + kSolveWarps + kPrepWarps);
        run_ctrl<kDiag>(cw, smem, mi, tmem, maps, p, n_chunks);
    }

    tc_fence_before();
    __syncthreads();
    if (mi.abort) {
        // a wait ran out: before the shared memory is given back, leave the copy engine time to land whatever this
        // CTA still has in flight (its loads complete in a microsecond or two), then report
        __nanosleep(20000);
        __syncthreads();
        if (tid == 0) atomicExch(p.status, 1u);
    }
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem));
}

// ---- host side ----------------------------------------------------------------------------------------

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

// [B][T][H][inner] tensor of bf16 (inner = 128) or fp32 (inner = 64), box = 64 tokens of one head.
bool make_map(CUtensorMap *map, const void *base, int B, int T, int H, bool f32 = false, bool half_swizzled = false)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t inner = f32 ? M : DV, row = 256;      // elements, bytes per (token, head)
    const cuuint64_t dims[4] = {inner, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)B};
    const cuuint64_t strides[3] = {row, (cuuint64_t)H * row, (cuuint64_t)T * H * row};
    // half_swizzled (outputs): a box is 64 tokens x 64 channels (128-byte rows) in the 128-byte swizzle
    const cuuint32_t box[4] = {(cuuint32_t)(half_swizzled ? inner / 2 : inner), 1, (cuuint32_t)C, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base),
              dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              half_swizzled ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// ---- scratch that nobody allocates -------------------------------------------------------------------
// The tensor-core kernel keeps its status word in caller-provided scratch.  For callers that cannot provide
// any, the same kernel can run on this statically allocated block instead: it is part of the library image,
// so every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// In host code `g_static_scratch` is only a handle, not a device address; the address has to be asked for,
// once per device, with that device current.
cudaError_t static_scratch_address(void **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_ptr[dev] = ptr;
    }
    *out = g_static_ptr[dev];
    return cudaSuccess;
}
}  // namespace

cudaError_t launch_forward_ws_static(const ForwardArgs &a, cudaStream_t stream, int *launches)
{
    void *scratch = nullptr;
    const cudaError_t e = static_scratch_address(&scratch);
    if (e != cudaSuccess) return e;
    // the block keeps whatever the last call left in it; the launcher clears the status word on the stream
    return launch_forward_ws(a, scratch, kStaticScratchBytes, stream, launches);
}

cudaError_t read_static_status(cudaStream_t stream, uint32_t *word)
{
    void *scratch = nullptr;
    cudaError_t e = static_scratch_address(&scratch);
    if (e != cudaSuccess) return e;
    e = cudaMemcpyAsync(word, scratch, sizeof(uint32_t), cudaMemcpyDeviceToHost, stream);
    if (e != cudaSuccess) return e;
    return cudaStreamSynchronize(stream);
}

// (B * H is bounded so that the unit cursor's quotients by multiplication stay exact.)
bool forward_ws_supported(const ForwardArgs &a)
{
    return a.dtype == 1 && a.d_k == DK && a.d_v == DV && a.chunk == C && (long long)a.B * a.H <= 16384;
}

// Scratch layout: [0, 256) status word; then, when the block is large enough for time slicing,
// [256, 256 + round256(4 BH)) slice counters and BH boundary states of d_k x d_v floats.
size_t forward_ws_scratch_bytes(int B, int H)
{
    const size_t bh = (size_t)B * H;
    return kWsMinScratchBytes + ((bh * 4 + 255) & ~(size_t)255) + bh * DK * DV * 4;
}

// How the launcher cuts BH sequences of NC chunks for a device of n_sm SMs (pure host arithmetic).
void forward_ws_partition(int BH, int NC, int n_sm, bool cuts_allowed, int *slices, int *balanced, double *periods)
{
    // Time slices per sequence: one CTA per SM works through ceil(units / SMs) units of NC / Q chunks.  More
    // slices even out the last round (256 sequences on 148 SMs: two rounds of 128 chunks, or seven rounds of
    // 32); every unit boundary costs about one chunk period (the state goes through global memory and the next
    // slice waits for it).  The smallest Q within 3 % of the cheapest is taken.
    // With at least as many sequences as SMs the balanced partition (equal contiguous ranges of the chunks of all
    // sequences, see ChunkCursor) has no last round at all and two boundaries per CTA at most.  Its chunks are
    // slower, though: measured per-CTA timelines show the two SMs of a TPC finishing together to the microsecond
    // and the kernel, bound by instruction fetch, running 5 to 23 % slower per chunk once the CTAs reach their
    // boundaries at different times and stop executing the same code in step (equal-sized slices keep them in
    // step).  So it is taken only when its chunk count, weighted by 1.25, is still the smaller: shapes the slices
    // cannot even out (odd chunk counts, short sequences), where it measured 21 to 22 % faster.
    int Q = 1, bal = 0;
    double best = (double)((BH + n_sm - 1) / n_sm) * (NC + 1.0);   // uncut: whole sequences, round after round
    if (cuts_allowed) {
        for (int q = 1; q <= 8; q *= 2) {
            if (NC % q != 0 || NC / q < 4) break;
            // the q slices of one sequence run one after another: never fewer than q unit times
            const long units = (long)BH * q, rounds = (units + n_sm - 1) / n_sm;
            const double cost = (double)(rounds > q ? rounds : q) * (NC / q + 1.0);
            if (q == 1 || cost < 0.97 * best) { best = cost; Q = q; }
        }
        const long long N = (long long)BH * NC;
        if (BH >= n_sm && NC >= 4 && N * NC < 0x100000000ll && 1.25 * ((double)((N + n_sm - 1) / n_sm) + 2.0) < best) {
            bal = 1;
            Q = 1;
            best = (double)((N + n_sm - 1) / n_sm) + 2.0;
        }
    }
    *slices = Q;
    *balanced = bal;
    if (periods) *periods = best;      // the schedule's length in chunk periods (what the choice was made on)
}

cudaError_t launch_forward_ws(const ForwardArgs &a, void *scratch, size_t scratch_bytes, cudaStream_t stream, int *launches,
                              bool clear_status)
{
    Maps maps;
    if (!make_map(&maps.v, a.v, a.B, a.T, a.H) || !make_map(&maps.o, a.o, a.B, a.T, a.H, false, true) ||
        !make_map(&maps.oim, a.o_im ? a.o_im : a.o, a.B, a.T, a.H, false, true) || !make_map(&maps.q, a.q, a.B, a.T, a.H) ||
        !make_map(&maps.k, a.k, a.B, a.T, a.H) || !make_map(&maps.al, a.alpha, a.B, a.T, a.H, true) ||
        !make_map(&maps.th, a.theta, a.B, a.T, a.H, true))
        return cudaErrorInvalidValue;
    const bool fused = a.fused != 0;
    // three instantiations: plain, raw inputs (stable parameterisation inside), and the diagnostic one whose waits
    // take their limit from the launch
    const bool diag = a.debug_withhold != 0 || a.wait_ticks != 0;
    if (diag && fused) return cudaErrorInvalidValue;
    const void *kernel = diag    ? reinterpret_cast<const void *>(sfda_forward_ws_kernel<false, true>)
                         : fused ? reinterpret_cast<const void *>(sfda_forward_ws_kernel<true, false>)
                                 : reinterpret_cast<const void *>(sfda_forward_ws_kernel<false, false>);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    int dev = 0, n_sm = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;

    const int BH = a.B * a.H, NC = (a.T + C - 1) / C;
    int Q = 1, bal = 0;
    forward_ws_partition(BH, NC, n_sm, scratch_bytes >= forward_ws_scratch_bytes(a.B, a.H), &Q, &bal, nullptr);
    if (a.debug_slices > 0) {      // diagnostic launches: the caller fixes the number of time slices
        if (NC % a.debug_slices != 0 || scratch_bytes < forward_ws_scratch_bytes(a.B, a.H)) return cudaErrorInvalidValue;
        Q = a.debug_slices;
        bal = 0;
    }
    const bool pieces = Q > 1 || bal;   // sequences are cut: counters and boundary states in use, CTAs wait on one another
    const size_t header = kWsMinScratchBytes + (pieces ? (((size_t)BH * 4 + 255) & ~(size_t)255) : 0);
    // The status word is only ever set by the kernel, never cleared: a caller that runs several launches on one
    // scratch block and reads the word once at the end clears it with the first launch only.
    if (clear_status)
        e = cudaMemsetAsync(scratch, 0, header, stream);
    else if (header > kWsMinScratchBytes)
        e = cudaMemsetAsync(static_cast<char *>(scratch) + kWsMinScratchBytes, 0, header - kWsMinScratchBytes, stream);
    if (e != cudaSuccess) return e;
    Params p;
    p.q = static_cast<const __nv_bfloat16 *>(a.q);
    p.k = static_cast<const __nv_bfloat16 *>(a.k);
    p.alpha = a.alpha;
    p.theta = a.theta;
    p.beta = a.beta;
    p.S0 = a.S0;
    p.S_T = a.S_T;
    p.phase_out = a.phase_turns;
    p.status = static_cast<uint32_t *>(scratch);
    p.flags = reinterpret_cast<uint32_t *>(static_cast<char *>(scratch) + kWsMinScratchBytes);
    p.handoff = reinterpret_cast<float *>(static_cast<char *>(scratch) + header);
    p.T = a.T;
    p.H = a.H;
    p.has_o_im = a.o_im != nullptr;
    p.wait_limit = a.wait_ticks ? a.wait_ticks : 0x80000000u;
    p.withhold = a.debug_withhold;
    p.BH = BH;
    p.Q = Q;
    p.U = NC / Q;
    p.n_units = BH * Q;
    p.magic_BH = BH > 1 ? (uint32_t)(0x100000000ull / (unsigned)BH) + 1u : 0u;
    p.magic_H = a.H > 1 ? (uint32_t)(0x100000000ull / (unsigned)a.H) + 1u : 0u;
    const unsigned grid = (unsigned)(p.n_units < n_sm ? p.n_units : n_sm);
    p.bal = bal;
    p.NC = NC;
    p.bal_base = (int)((long long)BH * NC / grid);
    p.bal_rem = (int)((long long)BH * NC % grid);
    p.magic_NC = NC > 1 ? (uint32_t)(0x100000000ull / (unsigned)NC) + 1u : 0u;
    p.a_lo = a.alpha_min;
    p.a_range = a.alpha_max - a.alpha_min;
    p.th_max = a.theta_max;
    p.th_m2 = -2.0f * a.theta_max;
    p.eps = a.eps;
    // With time slices a CTA waits for the CTA that runs the previous slice of its sequence, so all CTAs of the
    // launch have to be resident together: a cooperative launch makes the driver guarantee just that, whatever else
    // is running on other streams.  (Never more CTAs than SMs, one per SM: the grid always fits.)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = pieces ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    void *kargs[2] = {&maps, &p};
    e = cudaLaunchKernelExC(&cfg, kernel, kargs);
    if (e != cudaSuccess) return e;
    e = cudaGetLastError();
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace sfda
