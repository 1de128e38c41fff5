// PTX wrappers shared by the tensor-core kernels: mbarrier, TMA, tcgen05 (alloc-free parts), the
// shared-memory / instruction descriptors for bf16 K-major 128B-swizzled operands, TMEM load/store,
// and the warp-level tf32 MMA used by the triangular solve.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace sfda {
namespace tc {

constexpr uint32_t kSpinLimit = 1u << 22;

// ---- small PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bounded wait: returns false when the phase did not complete within the spin limit.
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, uint32_t parity)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok)
            : "r"(smem_u32(bar)), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, unsigned long long *bar, int c0, int c1,
                                            int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap *map, const void *src, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// K-major, 128-byte-swizzled operand tile: 8-row atoms of 1024 B (stride-dimension offset 1024).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// kind::f16 instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, M = 128.
__device__ __forceinline__ constexpr uint32_t idesc(int N, int neg_b)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)neg_b << 14) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t id, uint32_t acc)
{
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                 ::"r"(d), "l"(a), "l"(b), "r"(id), "r"(acc)
                 : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t b, uint32_t id, uint32_t acc)
{
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
                 ::"r"(d), "r"(a), "l"(b), "r"(id), "r"(acc)
                 : "memory");
}
// Same with the shared-memory descriptor given as its two 32-bit halves: advancing along K only changes the
// low half, so the issuing thread spends one 32-bit add per instruction.
__device__ __forceinline__ void mma_ts2(uint32_t d, uint32_t a, uint32_t b_lo, uint32_t b_hi, uint32_t id, uint32_t acc)
{
    asm volatile(
        "{\n.reg .pred p;\n.reg .b64 db;\nmov.b64 db, {%2, %3};\nsetp.ne.b32 p, %5, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n}\n" ::"r"(d),
        "r"(a), "r"(b_lo), "r"(b_hi), "r"(id), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void mma_ss2(uint32_t d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi, uint32_t id,
                                        uint32_t acc)
{
    asm volatile(
        "{\n.reg .pred p;\n.reg .b64 da, db;\nmov.b64 da, {%1, %2};\nmov.b64 db, {%3, %4};\nsetp.ne.b32 p, %6, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n}\n" ::"r"(d),
        "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(id), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void mma_commit(unsigned long long *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// K = 64 (one swizzle span) product: four K = 16 instructions. A from shared memory / from TMEM.
__device__ __forceinline__ void mma_k64_ss(uint32_t d, uint32_t a_saddr, uint32_t b_saddr, uint32_t id, bool acc)
{
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
        mma_ss(d, smem_desc(a_saddr + 32 * ks), smem_desc(b_saddr + 32 * ks), id, (acc || ks > 0) ? 1u : 0u);
}
__device__ __forceinline__ void mma_k64_ts(uint32_t d, uint32_t a_tmem, uint32_t b_saddr, uint32_t id, bool acc)
{
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) mma_ts(d, a_tmem + 8 * ks, smem_desc(b_saddr + 32 * ks), id, (acc || ks > 0) ? 1u : 0u);
}

#define SFDA_R32(r, o) \
    "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), "=r"(r[o + 6]), \
    "=r"(r[o + 7]), "=r"(r[o + 8]), "=r"(r[o + 9]), "=r"(r[o + 10]), "=r"(r[o + 11]), "=r"(r[o + 12]),               \
    "=r"(r[o + 13]), "=r"(r[o + 14]), "=r"(r[o + 15])
#define SFDA_W32(r, o) \
    "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), "r"(r[o + 6]), \
    "r"(r[o + 7]), "r"(r[o + 8]), "r"(r[o + 9]), "r"(r[o + 10]), "r"(r[o + 11]), "r"(r[o + 12]), "r"(r[o + 13]), \
    "r"(r[o + 14]), "r"(r[o + 15])

// 16 consecutive 32-bit columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t addr, uint32_t *r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : SFDA_R32(r, 0)
                 : "r"(addr));
}
__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t *r)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 ::"r"(addr), SFDA_W32(r, 0)
                 : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t addr, const uint32_t *r)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(addr), "r"(r[0]), "r"(r[1]),
                 "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t addr, uint32_t *r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(addr));
}
// 16 lanes x 64 columns of 32-bit tensor memory in the 16x256b fragment shape: for column block i (8 columns),
// thread T receives r[4i], r[4i+1] = (lane T / 4, columns 8i + 2 (T % 4), + 1) and r[4i+2], r[4i+3] = the same
// columns of lane T / 4 + 8 (the accumulator-fragment layout of the warp-level MMA).
__device__ __forceinline__ void tmem_ld_16x256b_x8(uint32_t addr, uint32_t *r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : SFDA_R32(r, 0), SFDA_R32(r, 16)
        : "r"(addr));
}
__device__ __forceinline__ void tmem_ld_16x256b_x4(uint32_t addr, uint32_t *r)
{
    asm volatile("tcgen05.ld.sync.aligned.16x256b.x4.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : SFDA_R32(r, 0)
                 : "r"(addr));
}
// Four 8 x 8 matrices of 16-bit elements, stored transposed: lane l gives the address of (transposed) row l % 8 of
// matrix l / 8; register k of thread T holds elements (row T / 4, columns 2 (T % 4), + 1) of matrix k.
__device__ __forceinline__ void stmatrix_x4_trans(uint32_t saddr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(saddr), "r"(a), "r"(b),
                 "r"(c), "r"(d)
                 : "memory");
}
__device__ __forceinline__ uint16_t lds16(uint32_t saddr)
{
    uint16_t v;
    asm volatile("ld.shared.b16 %0, [%1];" : "=h"(v) : "r"(saddr));
    return v;
}
// x + y for a bf16 x (its 16 bits as loaded) and an fp32 y, in one instruction (the bf16 is exact in fp32, so the
// result is the fp32 sum of the two)
__device__ __forceinline__ float add_bf16_f32(uint16_t x, float y)
{
    float r;
    asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(r) : "h"(x), "f"(y));
    return r;
}
template <int N>
__device__ __forceinline__ void tmem_ld(uint32_t addr, uint32_t *r)
{
#pragma unroll
    for (int i = 0; i < N; i += 16) tmem_ld16(addr + i, r + i);
}
template <int N>
__device__ __forceinline__ void tmem_st(uint32_t addr, const uint32_t *r)
{
#pragma unroll
    for (int i = 0; i < N; i += 16) tmem_st16(addr + i, r + i);
}

// Two floats -> packed bf16x2 (low half = lo), one conversion instruction.
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// Shared-memory stores / loads by 32-bit shared address (no 64-bit generic address arithmetic).
__device__ __forceinline__ void sts32(uint32_t saddr, uint32_t v)
{
    asm volatile("st.shared.b32 [%0], %1;" ::"r"(saddr), "r"(v) : "memory");
}
__device__ __forceinline__ void sts16(uint32_t saddr, uint16_t v)
{
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(saddr), "h"(v) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t saddr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(saddr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void sts64(uint32_t saddr, uint32_t a, uint32_t b)
{
    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(saddr), "r"(a), "r"(b) : "memory");
}
__device__ __forceinline__ uint32_t lds32(uint32_t saddr)
{
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(saddr));
    return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t saddr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(saddr));
    return v;
}
// Four 8 x 8 matrices of 16-bit elements = four 8-row x 4-column blocks of 32-bit elements: lane l supplies the
// 16-byte row address of row l % 8 of block l / 8; thread T receives element (T / 4, T % 4) of every block, which
// is the A-fragment layout of the m16n8k8 tf32 MMA when the blocks are (rows 0-7 | rows 8-15) x (k 0-3 | k 4-7).
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t saddr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(saddr));
}
// Global loads through the read-only path that only happen when `on` is set (the destination keeps its value
// otherwise): no branch, so neighbouring work can be scheduled across them.
__device__ __forceinline__ void ldg64_if(uint32_t &x, uint32_t &y, const void *ptr, bool on)
{
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %3, 0;\n@p ld.global.cg.v2.b32 {%0, %1}, [%2];\n}\n"
                 : "+r"(x), "+r"(y)
                 : "l"(ptr), "r"((uint32_t)on));
}
// Byte offset of element (row r, k-element e < 64) in a K-major 128B-swizzled tile.
__device__ __forceinline__ int sw_off(int r, int e)
{
    return (r >> 3) * 1024 + (r & 7) * 128 + ((((e >> 3) ^ r) & 7) << 4) + ((e & 7) << 1);
}
// ---- warp-level tf32 MMA used by the triangular solve ------------------------------------------------
// fp32 bits used directly as a tf32 operand: the tensor core ignores the low 13 mantissa bits (truncation,
// relative error below 2^-10), and no conversion instruction is spent.
__device__ __forceinline__ uint32_t to_tf32(float x) { return __float_as_uint(x); }
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2])
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
// (cr + i ci) += A[a_row0 .. +15][a_col0 + 8 s ..] * B[b_row0 + 8 s ..][b_col0 .. +7] over k-steps s in [s0, s1),
// complex fp32 matrices in shared memory (row strides a_ld, b_ld); one 16 x 8 output tile per warp.
__device__ __forceinline__ void cmma_16x8(float (&cr)[4], float (&ci)[4], const float *Ar, const float *Ai, int a_ld,
                                          int a_row0, int a_col0, const float *Br, const float *Bi, int b_ld,
                                          int b_row0, int b_col0, int s0, int s1, int lane)
{
    const int g = lane >> 2, tg = lane & 3;
#pragma unroll 1
    for (int s = s0; s < s1; ++s) {
        const int ao = (a_row0 + g) * a_ld + a_col0 + 8 * s + tg;
        uint32_t ar[4], ai[4], nai[4], br[2], bi[2];
        ar[0] = to_tf32(Ar[ao]);
        ar[1] = to_tf32(Ar[ao + 8 * a_ld]);
        ar[2] = to_tf32(Ar[ao + 4]);
        ar[3] = to_tf32(Ar[ao + 8 * a_ld + 4]);
        ai[0] = to_tf32(Ai[ao]);
        ai[1] = to_tf32(Ai[ao + 8 * a_ld]);
        ai[2] = to_tf32(Ai[ao + 4]);
        ai[3] = to_tf32(Ai[ao + 8 * a_ld + 4]);
#pragma unroll
        for (int x = 0; x < 4; ++x) nai[x] = ai[x] ^ 0x80000000u;
        const int bo = (b_row0 + 8 * s + tg) * b_ld + b_col0 + g;
        br[0] = to_tf32(Br[bo]);
        br[1] = to_tf32(Br[bo + 4 * b_ld]);
        bi[0] = to_tf32(Bi[bo]);
        bi[1] = to_tf32(Bi[bo + 4 * b_ld]);
        mma_tf32(cr, ar, br);
        mma_tf32(cr, nai, bi);
        mma_tf32(ci, ar, bi);
        mma_tf32(ci, ai, br);
    }
}
// Store a 16 x 8 accumulator tile (times `scale`) at rows row0.., columns col0.. of a complex fp32 matrix.
__device__ __forceinline__ void store_tile(const float (&cr)[4], const float (&ci)[4], float scale, float *Dr, float *Di,
                                           int ld, int row0, int col0, int lane)
{
    const int g = lane >> 2, tg = lane & 3;
    const int o = (row0 + g) * ld + col0 + 2 * tg;
    Dr[o] = scale * cr[0];
    Dr[o + 1] = scale * cr[1];
    Dr[o + 8 * ld] = scale * cr[2];
    Dr[o + 8 * ld + 1] = scale * cr[3];
    Di[o] = scale * ci[0];
    Di[o + 1] = scale * ci[1];
    Di[o + 8 * ld] = scale * ci[2];
    Di[o + 8 * ld + 1] = scale * ci[3];
}


}  // namespace tc
}  // namespace sfda
