// Tensor-core decode attention (MKV_DECODE_TENSOR): one-pass mixed-format split-KV scan.
//
// Section 3.3 / 4.1: every page of a request row is read in its own physical format (FP8 for
// Recent/Anchor, TQ3 for Stale), all tokens share one softmax, the whole GQA group reuses each
// unpacked tile, and split partials (m, l, O) are merged with Eq. (softmax-merge).
//
// Mapping to the hardware
//   * work = (request, KV head, page) triples in row-major order, cut into equal contiguous ranges,
//     one per block (persistent grid, a multiple of the SM count); a block processes the
//     (request, KV head) segments of its range one after another, its warps taking pages round-robin.
//   * each warp streams its pages through a private ring of shared-memory slots filled by bulk
//     asynchronous copies (cp.async.bulk + mbarrier), several pages ahead of the arithmetic.
//   * a 16-token page x d dims is exactly the A operand of m16n8k16 MMAs whose B operand is the
//     (rotated) query of the 8-column head group: S[16 tokens][8 heads] = K q^T.  TQ3 keys stay in
//     the rotated domain; the query is rotated instead (q' = d^-1/2 H (sigma . q)).  The packed
//     3-bit codes are stored in the register layout of that A fragment, so unpacking is a byte
//     table lookup (PRMT) per four codes for keys and one masked OR plus one half2 FMA per two
//     codes for values -- no shared-memory round trip, no dequantised tile.
//   * P = exp2(S - m) is transposed in registers (movmatrix) into the B operand of
//     O^T[16 channels][8 heads] += V^T P, one MMA per 16 channels; the row sums come from one more
//     MMA against a matrix of ones.  TQ3 values enter that MMA as their integer codes; the
//     per-channel fp16 scale and zero of the page are applied to the 16x8 result in fp32.
//   * partial results of a block that covers only part of a (request, KV head) row go to the
//     workspace; the last block to arrive for that row (atomic ticket) merges them.  Nothing spins
//     on another block.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <math_constants.h>

#include <cstdlib>

#include "mkv_internal.cuh"

namespace mkv {

constexpr int kMaxCtas = 512;        // upper bound of the persistent grid (sizes the workspace)
constexpr int kMaxBatch = 1024;      // requests per call
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleSlack = 8.0f;   // running maximum is only raised when exceeded by 2^8

size_t decode_ws_tensor_bytes(int, int, int, int d)
{
    return (size_t)2 * kMaxCtas * (8 * d + 16) * sizeof(float);
}

struct DecodeParams {
    const uint8_t* fp8;
    const uint8_t* tq3;
    int fp8_pages, tq3_pages, hkv, group;
    float k_scale, v_scale;
    SigmaBits sigma;
    const __nv_bfloat16* q;
    const int32_t* bt;
    const uint8_t* tags;
    const int32_t* lens;
    int B, max_pages;
    float scale;
    float* out;
    float* lse;
    uint32_t* tickets;     // [B * hkv], zero on entry, zero on exit
    float* partials;       // [2 * grid][8*D + 16]
    uint32_t* status;
};

// ------------------------------------------------------------------------------------------------
// small PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t s)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(s));
    return r;
}

// (a & b) | c in one LOP3
__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}

__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// same product with a zero accumulator: d = A B
__device__ __forceinline__ void mma16816_zero(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x)
{
    uint32_t r;
    asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(r) : "r"(x));
    return r;
}

__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint16_t v)
{
    uint32_t r;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(v));
    return r;
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

__device__ __forceinline__ uint32_t hfma2_u32(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t r;
    asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// bulk asynchronous copy global -> this block's shared memory, completion counted on an mbarrier
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ uint2 lds64(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}

__device__ __forceinline__ uint16_t lds16(uint32_t addr)
{
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}

// ------------------------------------------------------------------------------------------------
// TQ3 unpack
// ------------------------------------------------------------------------------------------------
// Four 3-bit key codes in the four low nibbles of `sel` (bit 3 of each nibble clear) -> two half2
// registers holding the signed fp16 codebook levels.  The two byte tables hold the high and the low
// bytes of {+C0,+C1,+C2,+C3,-C0,-C1,-C2,-C3} = fp16 {33D8, 3A0C, 3D60, 404E | sign}.
__device__ __forceinline__ void key_lut4(uint32_t sel, uint32_t& r0, uint32_t& r1)
{
    const uint32_t hi = prmt(0x403D3A33u, 0xC0BDBAB3u, sel);
    const uint32_t lo = prmt(0x4E600CD8u, 0x4E600CD8u, sel);
    r0 = prmt(lo, hi, 0x5140u);
    r1 = prmt(lo, hi, 0x7362u);
}

// Two 3-bit value codes sitting at bit POS of each 16-bit half of x -> half2 of the integer codes.
// (x & mask) | 0x6400 is the fp16 number 1024 + code * 2^POS; one FMA recovers the code exactly.
// The per-channel scale and zero are applied in fp32 after the token sum:
//   sum_t p_t (scale*code_t + zero) = scale * (sum_t p_t code_t) + zero * (sum_t p_t).
template <int POS>
__device__ __forceinline__ uint32_t value_code(uint32_t x)
{
    constexpr uint32_t mask = 0x00070007u << POS;
    const uint32_t u = lop3_and_or(x, mask, 0x64006400u);
    // 2^-POS and -1024 * 2^-POS as fp16 bit patterns (exponent arithmetic on 1.0 = 0x3C00, -1024 = 0xE400)
    constexpr uint32_t mul = (0x3C00u - (POS << 10)) * 0x00010001u;
    constexpr uint32_t add = (0xE400u - (POS << 10)) * 0x00010001u;
    return hfma2_u32(u, mul, add);
}

__device__ __forceinline__ float2 half2_to_float2(uint32_t x)
{
    return __half22float2(*reinterpret_cast<const __half2*>(&x));
}

// acc[channel rows g, g+8][heads] += scale_row * t + zero_row * psum_head
__device__ __forceinline__ void affine_accumulate(float (&acc)[4], const float (&t)[4], uint32_t sc_pair, uint32_t zp_pair,
                                                  float ps0, float ps1)
{
    const float2 sc = half2_to_float2(sc_pair), zp = half2_to_float2(zp_pair);
    acc[0] = fmaf(sc.x, t[0], fmaf(zp.x, ps0, acc[0]));
    acc[1] = fmaf(sc.x, t[1], fmaf(zp.x, ps1, acc[1]));
    acc[2] = fmaf(sc.y, t[2], fmaf(zp.y, ps0, acc[2]));
    acc[3] = fmaf(sc.y, t[3], fmaf(zp.y, ps1, acc[3]));
}

// ------------------------------------------------------------------------------------------------
// kernel
// ------------------------------------------------------------------------------------------------
// NW warps form NU = NW / HALVES units.  A unit owns a ring and processes one page at a time; with
// HALVES == 2 the two warps of a unit split the head dimension (key blocks for the scores, channel
// blocks for the output), exchange their partial scores through shared memory and each keep half of
// the accumulators, which halves the registers per thread.
template <int D, int NW, int NSTAGE, int HALVES>
struct Geo {
    static constexpr int NU = NW / HALVES;
    static constexpr int NB = D / 16;                       // 16-wide blocks along d
    static constexpr int LW = 3 * NB / 4;                   // packed words per lane and code section
    static constexpr int TQ3_REC = 16 * D + 32;
    static constexpr int FP8_HALF = 16 * D;
    static constexpr int SLOT = (TQ3_REC + 127) / 128 * 128;
    static constexpr int RING = NU * NSTAGE * SLOT;
    static constexpr int QFRAG = NB * 32 * 8;               // one set of query B fragments
    static constexpr int OFF_QT = RING;
    static constexpr int OFF_QL = OFF_QT + QFRAG;            // low-order halves of the rotated query
    static constexpr int OFF_QF = OFF_QL + QFRAG;
    static constexpr int OFF_BAR = OFF_QF + QFRAG;
    static constexpr int OFF_XCH = OFF_BAR + NU * NSTAGE * 8;   // [unit][parity][half][lane] float4
    static constexpr int OFF_CUM = OFF_XCH + NU * 2 * 2 * 512;
    static constexpr int OFF_STRIDE = OFF_CUM + (kMaxBatch + 1) * 4;
    static constexpr int OFF_M = OFF_STRIDE + kMaxBatch * 4;
    static constexpr int OFF_L = OFF_M + NW * 8 * 4;
    static constexpr int OFF_FLAG = OFF_L + NW * 8 * 4;
    static constexpr int SMEM = OFF_FLAG + 16;
    static_assert(HALVES == 1 || (HALVES == 2 && D == 256), "the head dimension is split only for d = 256");
    static_assert(HALVES == 1 || NSTAGE == 4, "a two-warp unit returns slots one page late: an FP8 page needs 2 + 2 slots");
    static_assert(NW >= 8, "one warp per column of the 8-wide head group builds the query fragments");
    static_assert(NSTAGE == 2 || NSTAGE == 4, "ring positions are taken modulo a power of two; an FP8 page takes two slots");
    static_assert(NSTAGE * SLOT >= 8 * D * 4, "ring doubles as the cross-warp reduction buffer");
    static_assert(FP8_HALF <= SLOT, "half an FP8 record fits a slot");
    static_assert(RING >= kMaxCtas * 4 + 2 * kMaxCtas * 8 * 4, "ring doubles as the final-merge scratch");
};

#ifdef MKV_TIMELINE
// profiling build only: thread 0 of every block accumulates the time spent in each phase
__device__ unsigned long long g_timeline[kMaxCtas * 16];
__device__ __forceinline__ unsigned long long tl_now()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define MKV_STAMP(k)                                                      \
    do {                                                                  \
        if (threadIdx.x == 0) {                                            \
            const unsigned long long t__ = tl_now();                      \
            if ((k) == 0) { g_timeline[blockIdx.x * 16 + 15] = t__; for (int z__ = 0; z__ < 15; ++z__) g_timeline[blockIdx.x * 16 + z__] = 0; } \
            else g_timeline[blockIdx.x * 16 + (k)] += t__ - tl_last;       \
            tl_last = t__;                                                \
            g_timeline[blockIdx.x * 16 + 14] = t__;                        \
        }                                                                 \
    } while (0)
#else
#define MKV_STAMP(k)
#endif

// Running state of one warp for one (request, KV head) segment: O^T accumulators [d channels x 8
// heads] in the MMA C layout, row sums and the (lazily raised) running maximum of the two head
// columns this lane owns, all in log2 units.
template <int NB>
struct WarpAcc {
    float o[NB][4];
    float l[2];
    float m[2];
};

// Scores of one page -> probabilities.  s[0..1] = token g, s[2..3] = token g+8 (heads 2tq, 2tq+1).
// Updates the running maximum (only when it is exceeded by more than 2^kRescaleSlack, so that
// accumulators are rarely rescaled), and returns P^T as MMA B fragments split into an fp16 pair
// hi (pb) + lo (pc), plus the page's row sums ps[0..1].
template <int NB>
__device__ __forceinline__ void softmax_page(WarpAcc<NB>& acc, const float (&s)[4], uint32_t& pb0, uint32_t& pb1,
                                             uint32_t& pc0, uint32_t& pc1, float (&ps)[4])
{
    constexpr uint32_t FULL = 0xffffffffu;
    float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(FULL, mx0, o));
        mx1 = fmaxf(mx1, __shfl_xor_sync(FULL, mx1, o));
    }
    const bool up0 = mx0 > acc.m[0] + kRescaleSlack, up1 = mx1 > acc.m[1] + kRescaleSlack;
    if (__any_sync(FULL, up0 || up1)) {
        const float f0 = up0 ? fast_exp2(acc.m[0] - mx0) : 1.f, f1 = up1 ? fast_exp2(acc.m[1] - mx1) : 1.f;
        if (up0) acc.m[0] = mx0;
        if (up1) acc.m[1] = mx1;
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            acc.o[i][0] *= f0; acc.o[i][2] *= f0;
            acc.o[i][1] *= f1; acc.o[i][3] *= f1;
        }
        acc.l[0] *= f0;
        acc.l[1] *= f1;
    }
    const float p0 = fast_exp2(s[0] - acc.m[0]), p1 = fast_exp2(s[1] - acc.m[1]);
    const float p2 = fast_exp2(s[2] - acc.m[0]), p3 = fast_exp2(s[3] - acc.m[1]);
    const uint32_t ph01 = pack_f16x2(p0, p1), ph23 = pack_f16x2(p2, p3);
    const float2 h01 = half2_to_float2(ph01), h23 = half2_to_float2(ph23);
    pb0 = movmatrix_trans(ph01);
    pb1 = movmatrix_trans(ph23);
    pc0 = movmatrix_trans(pack_f16x2(p0 - h01.x, p1 - h01.y));
    pc1 = movmatrix_trans(pack_f16x2(p2 - h23.x, p3 - h23.y));
    // row sums through the tensor core: the same P that multiplies V
    const uint32_t ones[4] = {0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u};
    mma16816_zero(ps, ones, pb0, pb1);
    mma16816(ps, ones, pc0, pc1);
    acc.l[0] += ps[0];
    acc.l[1] += ps[1];
}

// The packed words of one lane for one code section: all of them (HALVES == 1) or the half that
// belongs to warp half hf (d = 256: words 0..5 or 6..11 of the lane's 12).
template <int D, int HALVES>
__device__ __forceinline__ void load_lane_words(uint32_t sec, int lane, int hf, uint32_t (&w)[3 * (D / 16) / 4 / HALVES])
{
    constexpr int LW = 3 * (D / 16) / 4;
    if constexpr (HALVES == 1) {
#pragma unroll
        for (int c = 0; c < LW / 4; ++c) {
            const uint4 v = lds128(sec + c * 512 + lane * 16);
            w[4 * c] = v.x; w[4 * c + 1] = v.y; w[4 * c + 2] = v.z; w[4 * c + 3] = v.w;
        }
        if constexpr (LW % 4 != 0) {
            const uint2 v = lds64(sec + (LW / 4) * 512 + lane * 8);
            w[LW - 2] = v.x; w[LW - 1] = v.y;
        }
    } else {
        if (hf == 0) {
            const uint4 v = lds128(sec + lane * 16);
            const uint2 u = lds64(sec + 512 + lane * 16);
            w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w; w[4] = u.x; w[5] = u.y;
        } else {
            const uint2 u = lds64(sec + 512 + lane * 16 + 8);
            const uint4 v = lds128(sec + 1024 + lane * 16);
            w[0] = u.x; w[1] = u.y; w[2] = v.x; w[3] = v.y; w[4] = v.z; w[5] = v.w;
        }
    }
}

// Pair exchange of partial scores (HALVES == 2): each warp stores its four partial sums, the two
// warps meet at their named barrier, and both form the same total.
struct PairCtx {
    uint32_t xch;       // shared address of this unit's exchange area [parity][half][lane] float4
    int bar_id;         // named barrier of the unit
    int hf;             // which half this warp is
    uint32_t parity;    // toggles every page
};

template <int HALVES>
__device__ __forceinline__ void pair_sum(float (&S)[4], PairCtx& px, int lane)
{
    if constexpr (HALVES == 2) {
        const uint32_t mine = px.xch + ((px.parity * 2 + px.hf) * 32 + lane) * 16;
        const uint32_t other = px.xch + ((px.parity * 2 + (px.hf ^ 1)) * 32 + lane) * 16;
        asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(mine), "f"(S[0]), "f"(S[1]), "f"(S[2]), "f"(S[3]) : "memory");
        asm volatile("bar.sync %0, 64;" ::"r"(px.bar_id) : "memory");
        float o0, o1, o2, o3;
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(o0), "=f"(o1), "=f"(o2), "=f"(o3) : "r"(other));
        S[0] += o0; S[1] += o1; S[2] += o2; S[3] += o3;
        px.parity ^= 1u;
    }
}

// One Stale page: record at shared address rec (key codes, value codes, g, scale/zero).
template <int D, int HALVES>
__device__ __forceinline__ void tq3_page(WarpAcc<D / 16 / HALVES>& acc, uint32_t rec, uint32_t qt_lane, float sc2, int lane,
                                         PairCtx& px)
{
    constexpr int NB = D / 16, NBH = NB / HALVES, LWH = 3 * NB / 4 / HALVES, NT = NB / 4 / HALVES, QFRAG = NB * 32 * 8;
    const int g = lane >> 2;
    const int j0 = HALVES == 2 ? px.hf * NT : 0;     // first word triple / block quad of this warp
    // ---- S = K q'^T
    float S0[4] = {0.f, 0.f, 0.f, 0.f}, S1[4] = {0.f, 0.f, 0.f, 0.f};
    {
        uint32_t kw[LWH];
        load_lane_words<D, HALVES>(rec, lane, px.hf, kw);
        const uint32_t qt_half = qt_lane + j0 * 4 * 256;
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            const uint32_t A = kw[3 * j], Bw = kw[3 * j + 1], Cw = kw[3 * j + 2];
            uint32_t sel[4];
            sel[0] = A & 0x77777777u;
            sel[1] = Bw & 0x77777777u;
            sel[2] = lop3_and_or(A >> 1, 0x44444444u, Cw & 0x33333333u);
            sel[3] = lop3_and_or(Bw >> 1, 0x44444444u, (Cw >> 2) & 0x33333333u);
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                uint32_t a[4];
                key_lut4(sel[w], a[0], a[1]);
                key_lut4(sel[w] >> 16, a[2], a[3]);
                const uint2 qv = lds64(qt_half + (4 * j + w) * 256);
                const uint2 qw = lds64(qt_half + QFRAG + (4 * j + w) * 256);
                if (w & 1) { mma16816(S1, a, qv.x, qv.y); mma16816(S1, a, qw.x, qw.y); }
                else       { mma16816(S0, a, qv.x, qv.y); mma16816(S0, a, qw.x, qw.y); }
            }
        }
    }
    float St[4] = {S0[0] + S1[0], S0[1] + S1[1], S0[2] + S1[2], S0[3] + S1[3]};
    pair_sum<HALVES>(St, px, lane);
    const uint32_t gaddr = rec + 12 * D;
    const float r0 = __half2float(__ushort_as_half(lds16(gaddr + 2 * g))) * sc2;
    const float r1 = __half2float(__ushort_as_half(lds16(gaddr + 2 * g + 16))) * sc2;
    const float s[4] = {St[0] * r0, St[1] * r0, St[2] * r1, St[3] * r1};
    uint32_t pb0, pb1, pc0, pc1;
    float ps[4];
    softmax_page<NBH>(acc, s, pb0, pb1, pc0, pc1, ps);

    // ---- O^T += V^T P with integer codes; scale and zero applied to the 16x8 result in fp32
    uint32_t vw[LWH];
    load_lane_words<D, HALVES>(rec + 6 * D, lane, px.hf, vw);
    const uint32_t meta = rec + 12 * D + 32 + g * 16 + j0 * 2 * 128;
#pragma unroll
    for (int j = 0; j < NT; ++j) {
        const uint32_t W0 = vw[3 * j], W1 = vw[3 * j + 1], W2 = vw[3 * j + 2];
        float t[4];
        uint32_t a[4];
        {   // blocks 4j, 4j+1
            const uint4 mt = lds128(meta + (2 * j) * 128);
            const uint32_t X1 = prmt(W0, W1, 0x6341u);
            a[0] = value_code<0>(W0);
            a[1] = value_code<3>(W0);
            a[2] = value_code<6>(W0);
            a[3] = value_code<1>(X1);
            mma16816_zero(t, a, pb0, pb1);
            mma16816(t, a, pc0, pc1);
            affine_accumulate(acc.o[4 * j], t, mt.x, mt.y, ps[0], ps[1]);
            a[0] = value_code<4>(X1);
            a[1] = value_code<7>(X1);
            a[2] = value_code<2>(W1);
            a[3] = value_code<5>(W1);
            mma16816_zero(t, a, pb0, pb1);
            mma16816(t, a, pc0, pc1);
            affine_accumulate(acc.o[4 * j + 1], t, mt.z, mt.w, ps[0], ps[1]);
        }
        {   // blocks 4j+2, 4j+3
            const uint4 mt = lds128(meta + (2 * j + 1) * 128);
            const uint32_t X0 = prmt(W1, W2, 0x6341u), X2 = W2 >> 8;
            a[0] = value_code<0>(X0);
            a[1] = value_code<3>(X0);
            a[2] = value_code<6>(X0);
            a[3] = value_code<1>(W2);
            mma16816_zero(t, a, pb0, pb1);
            mma16816(t, a, pc0, pc1);
            affine_accumulate(acc.o[4 * j + 2], t, mt.x, mt.y, ps[0], ps[1]);
            a[0] = value_code<4>(W2);
            a[1] = value_code<7>(W2);
            a[2] = value_code<2>(X2);
            a[3] = value_code<5>(X2);
            mma16816_zero(t, a, pb0, pb1);
            mma16816(t, a, pc0, pc1);
            affine_accumulate(acc.o[4 * j + 3], t, mt.z, mt.w, ps[0], ps[1]);
        }
    }
}

// One Recent/Anchor page: keys [16 tokens][d] e4m3 at kaddr, values [d channels][16 tokens] at vaddr.
template <int D, int HALVES>
__device__ __forceinline__ void fp8_page(WarpAcc<D / 16 / HALVES>& acc, uint32_t kaddr, uint32_t vaddr, uint32_t qf_lane,
                                         float score_scale, float v_scale, int valid, int lane, PairCtx& px)
{
    constexpr int NB = D / 16, NBH = NB / HALVES, NJ = D / 64 / HALVES;
    const int g = lane >> 2, tq = lane & 3;
    const int jj0 = HALVES == 2 ? px.hf * NJ : 0, cb0 = HALVES == 2 ? px.hf * NBH : 0;
    float S0[4] = {0.f, 0.f, 0.f, 0.f}, S1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int jl = 0; jl < NJ; ++jl) {
        const int j = jj0 + jl;
        const uint4 r0 = lds128(kaddr + g * D + 64 * j + 16 * tq);
        const uint4 r1 = lds128(kaddr + (g + 8) * D + 64 * j + 16 * tq);
        const uint32_t w0[4] = {r0.x, r0.y, r0.z, r0.w}, w1[4] = {r1.x, r1.y, r1.z, r1.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            uint32_t a[4];
            a[0] = e4m3x2_to_f16x2((uint16_t)(w0[w] & 0xFFFFu));
            a[1] = e4m3x2_to_f16x2((uint16_t)(w1[w] & 0xFFFFu));
            a[2] = e4m3x2_to_f16x2((uint16_t)(w0[w] >> 16));
            a[3] = e4m3x2_to_f16x2((uint16_t)(w1[w] >> 16));
            const uint2 qv = lds64(qf_lane + (4 * j + w) * 256);
            if (w & 1) mma16816(S1, a, qv.x, qv.y);
            else       mma16816(S0, a, qv.x, qv.y);
        }
    }
    float St[4] = {S0[0] + S1[0], S0[1] + S1[1], S0[2] + S1[2], S0[3] + S1[3]};
    pair_sum<HALVES>(St, px, lane);
    float s[4] = {St[0] * score_scale, St[1] * score_scale, St[2] * score_scale, St[3] * score_scale};
    // bytes of tokens beyond the sequence end are cleared so that stale NaN patterns cannot leak
    uint32_t keep_lo = 0xFFFFu, keep_hi = 0xFFFFu;   // byte masks for tokens (2tq,2tq+1), (2tq+8,2tq+9)
    if (valid < kPage) {
        if (g >= valid) s[0] = s[1] = -CUDART_INF_F;
        if (g + 8 >= valid) s[2] = s[3] = -CUDART_INF_F;
        keep_lo = (2 * tq < valid ? 0x00FFu : 0u) | (2 * tq + 1 < valid ? 0xFF00u : 0u);
        keep_hi = (2 * tq + 8 < valid ? 0x00FFu : 0u) | (2 * tq + 9 < valid ? 0xFF00u : 0u);
    }
    uint32_t pb0, pb1, pc0, pc1;
    float ps[4];
    softmax_page<NBH>(acc, s, pb0, pb1, pc0, pc1, ps);
    const bool scale_v = v_scale != 1.0f;
#pragma unroll
    for (int cb = 0; cb < NBH; ++cb) {
        const uint32_t r0 = vaddr + (16 * (cb0 + cb) + g) * 16 + 2 * tq, r1 = r0 + 8 * 16;
        uint32_t a[4];
        a[0] = e4m3x2_to_f16x2((uint16_t)(lds16(r0) & keep_lo));
        a[1] = e4m3x2_to_f16x2((uint16_t)(lds16(r1) & keep_lo));
        a[2] = e4m3x2_to_f16x2((uint16_t)(lds16(r0 + 8) & keep_hi));
        a[3] = e4m3x2_to_f16x2((uint16_t)(lds16(r1 + 8) & keep_hi));
        if (scale_v) {
            float t[4];
            mma16816_zero(t, a, pb0, pb1);
            mma16816(t, a, pc0, pc1);
#pragma unroll
            for (int e = 0; e < 4; ++e) acc.o[cb][e] = fmaf(v_scale, t[e], acc.o[cb][e]);
        } else {
            mma16816(acc.o[cb], a, pb0, pb1);
            mma16816(acc.o[cb], a, pc0, pc1);
        }
    }
}

template <int D, int NW, int NSTAGE, int MINB, int HALVES>
__global__ void __launch_bounds__(NW * 32, MINB) decode_tensor_kernel(const DecodeParams P)
{
#ifdef MKV_TIMELINE
    unsigned long long tl_last = 0;
#endif
    MKV_STAMP(0);
    using G = Geo<D, NW, NSTAGE, HALVES>;
    constexpr int NB = G::NB, NBH = NB / HALVES, NU = G::NU;
    constexpr uint32_t FULL = 0xffffffffu;
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    int* cum = reinterpret_cast<int*>(smem + G::OFF_CUM);
    int* strides = reinterpret_cast<int*>(smem + G::OFF_STRIDE);
    float* sm_m = reinterpret_cast<float*>(smem + G::OFF_M);
    float* sm_l = reinterpret_cast<float*>(smem + G::OFF_L);
    int* sm_flag = reinterpret_cast<int*>(smem + G::OFF_FLAG);
    float* red = reinterpret_cast<float*>(smem);            // [NU][D][8] over the ring, between segments

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    const int unit = warp / HALVES, hf = warp % HALVES;
    const int hkv = P.hkv, GQ = P.group, hq = hkv * GQ;

    // ---- prologue: barriers, zero rows of empty requests, prefix of pages -----------------------
    if (tid == 0) {
        for (int i = 0; i < NU * NSTAGE; ++i) mbar_init(sbase + G::OFF_BAR + 8 * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int b = blockIdx.x; b < P.B; b += gridDim.x)
        if (P.lens[b] <= 0) {
            for (int i = tid; i < hq * D; i += NW * 32) P.out[(size_t)b * hq * D + i] = 0.f;
            if (P.lse)
                for (int i = tid; i < hq; i += NW * 32) P.lse[(size_t)b * hq + i] = -CUDART_INF_F;
        }
    if (warp == 0) {
        int run = 0;
        for (int b0 = 0; b0 < P.B; b0 += 32) {
            const int b = b0 + lane;
            int n = 0;
            if (b < P.B) {
                const int len = P.lens[b];
                n = len > 0 ? ((len + kPage - 1) / kPage) * hkv : 0;
            }
            int inc = n;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(FULL, inc, o);
                if (lane >= o) inc += v;
            }
            if (b < P.B) cum[b] = run + inc - n;
            run += __shfl_sync(FULL, inc, 31);
        }
        if (lane == 0) cum[P.B] = run;
    } else {
        // Pages of a row are visited in a strided order, page(i) = i * stride mod n_pages, the stride
        // coprime to n_pages and near 0.618 n_pages: every contiguous range of positions then holds the
        // row's FP8 and TQ3 pages in their overall proportion, so equal ranges cost equal time.
        for (int b = tid - 32; b < P.B; b += NW * 32 - 32) {
            const int len = P.lens[b], n = (len + kPage - 1) / kPage;
            int st = (int)((float)n * 0.6180339f);
            if (st < 1) st = 1;
            for (; n > 1; ++st) {
                int a = st, c = n;
                while (c) { const int t = a % c; a = c; c = t; }
                if (a == 1) break;
            }
            strides[b] = st;
        }
    }
    __syncthreads();
    const long long W = cum[P.B];
    const int C = (int)(W < (long long)gridDim.x ? W : (long long)gridDim.x);   // blocks that get work
    if ((int)blockIdx.x >= C) return;
    auto range_start = [&](int c) -> int { return (int)((W * c) / C); };
    auto block_of = [&](int x) -> int {      // the block whose range holds linear index x
        int c = (int)(((long long)x * C) / W);
        while (c + 1 < C && range_start(c + 1) <= x) ++c;
        while (c > 0 && range_start(c) > x) --c;
        return c;
    };
    const int my_start = range_start(blockIdx.x), my_end = range_start(blockIdx.x + 1);

    // per-unit ring of NSTAGE slots: fill and drain positions, slots in flight, and one bit per slot with
    // the mbarrier phase the next wait on it must see (flipped every time the slot is consumed); with two
    // warps per unit both keep the same state and the first one issues the copies
    uint32_t head = 0, tail = 0, in_flight = 0, phase = 0;
    bool failed = false;
    const uint32_t ring = sbase + unit * NSTAGE * G::SLOT;
    const uint32_t bars = sbase + G::OFF_BAR + unit * NSTAGE * 8;
    PairCtx px;
    px.xch = sbase + G::OFF_XCH + unit * 2048;
    px.bar_id = 1 + unit;
    px.hf = hf;
    px.parity = 0;
    const bool issuer = (hf == 0) && (lane == 0);
    auto unit_sync = [&]() {
        if constexpr (HALVES == 2) asm volatile("bar.sync %0, 64;" ::"r"(px.bar_id) : "memory");
        else __syncwarp();
    };
    const uint32_t qt_lane = sbase + G::OFF_QT + lane * 8, qf_lane = sbase + G::OFF_QF + lane * 8;
    const float sc2 = P.scale * kLog2e;      // scores are kept in log2 units
    // bounded wait for ring slot s, then flip its expected phase
    auto wait_slot = [&](uint32_t s) {
        const uint32_t bar = bars + 8 * s, parity = (phase >> s) & 1u;
        phase ^= 1u << s;
        if (!mbar_try_wait(bar, parity)) {
            // give up after ~20 ms of wall time: flag the pool's status word and skip the remaining pages
            unsigned long long t0, t1;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
            int spins = 0;
            while (!mbar_try_wait(bar, parity)) {
                if ((++spins & 255) == 0) {
                    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
                    if (t1 - t0 > 20000000ull) {
                        failed = true;
                        atomicOr(P.status, kStTimeout);
                        break;
                    }
                }
            }
        }
        failed = __any_sync(FULL, failed);
    };

    int pos = my_start;
    int b = 0;
    MKV_STAMP(1);
    while (pos < my_end) {
        // ---- locate the segment: request b, KV head h, pages [pg0, pg0 + n_seg) ---------------
        while (cum[b + 1] <= pos) ++b;
        const int len = P.lens[b], n_pages = (len + kPage - 1) / kPage;
        const int h = (pos - cum[b]) / n_pages, pg0 = (pos - cum[b]) % n_pages;
        const int row_start = cum[b] + h * n_pages, row_end = row_start + n_pages;
        const int n_seg = min(my_end, row_end) - pos;
        const int32_t* bt_row = P.bt + (size_t)b * P.max_pages;
        const uint8_t* tag_row = P.tags + (size_t)b * P.max_pages;
        const int n_my = unit < n_seg ? (n_seg - unit + NU - 1) / NU : 0;   // this unit's pages, round-robin
        const int stride = strides[b];
        constexpr int EPL = D / 32;
        float qx[EPL];            // this warp's query head (warps 0..7), loaded before anything else waits
#pragma unroll
        for (int r = 0; r < EPL; ++r)
            qx[r] = (warp < GQ) ? __bfloat162float(P.q[((size_t)b * hq + h * GQ + warp) * D + lane * EPL + r]) : 0.f;
        auto page_at = [&](int i) -> int { return (int)(((unsigned)(pg0 + i) * (unsigned)stride) % (unsigned)n_pages); };

        // A walker enumerates, in order, the warp's pages of one format: 32 table entries at a time are
        // loaded (entry i in lane i) and the matching ones are visited through a ballot mask.
        struct Walker {
            int chunk;
            uint32_t mask;
            int id;
        };
        auto walker_load = [&](Walker& w, int want_tq3) {
            const int i = w.chunk * 32 + lane;
            int kind = 0;
            w.id = 0;
            if (i < n_my) {
                const int pg = page_at(unit + NU * i);
                const int id = bt_row[pg], tag = tag_row[pg];
                const int valid = min(kPage, len - pg * kPage);
                if (tag == MKV_TAG_STALE)
                    kind = (id >= 0 && id < P.tq3_pages && valid == kPage) ? 1 : 0;
                else
                    kind = (tag <= MKV_TAG_ANCHOR && id >= 0 && id < P.fp8_pages) ? 2 : 0;
                if (kind == 0 && want_tq3 && hf == 0) atomicOr(P.status, kStBounds);    // flagged once (first pass)
                w.id = id;
            }
            w.mask = __ballot_sync(FULL, kind == (want_tq3 ? 1 : 2));
        };
        // next matching page: returns false at the end; j = index inside the chunk
        auto walker_next = [&](Walker& w, int want_tq3, int& id, int& index) -> bool {
            while (w.mask == 0) {
                if ((w.chunk + 1) * 32 >= n_my) return false;
                ++w.chunk;
                walker_load(w, want_tq3);
            }
            const int j = __ffs(w.mask) - 1;
            w.mask &= w.mask - 1;
            id = __shfl_sync(FULL, w.id, j);
            index = w.chunk * 32 + j;
            return true;
        };

        WarpAcc<NBH> acc;
#pragma unroll
        for (int i = 0; i < NBH; ++i) acc.o[i][0] = acc.o[i][1] = acc.o[i][2] = acc.o[i][3] = 0.f;
        acc.l[0] = acc.l[1] = 0.f;
        acc.m[0] = acc.m[1] = -CUDART_INF_F;

        // ---- pass over the Stale (TQ3) pages: start the copies, then build the query fragments -----
        head = tail = 0;
        Walker prod, cons;
        prod.chunk = cons.chunk = 0;
        prod.mask = cons.mask = 0;
        prod.id = cons.id = 0;
        bool prod_more = n_my > 0;
        if (n_my > 0) {
            walker_load(prod, 1);
            cons = prod;
        }
        auto produce_tq3 = [&]() {
            while (prod_more && !failed && in_flight < NSTAGE) {
                int id, index;
                prod_more = walker_next(prod, 1, id, index);
                if (!prod_more) break;
                if (issuer) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    mbar_expect_tx(bars + 8 * head, G::TQ3_REC);
                    bulk_load(ring + head * G::SLOT, P.tq3 + ((size_t)id * hkv + h) * G::TQ3_REC, G::TQ3_REC, bars + 8 * head);
                }
                head = (head + 1) & (NSTAGE - 1);
                ++in_flight;
            }
        };
        produce_tq3();

        // query fragments: warp hd < 8 rotates head hd (loads were issued before the copies started)
        if (warp < 8) {
            const int hd = warp;
            float a[EPL];
#pragma unroll
            for (int r = 0; r < EPL; ++r) {
                const int i = lane * EPL + r;
                a[r] = ((P.sigma.w[i >> 5] >> (i & 31)) & 1u) ? -qx[r] : qx[r];
            }
#pragma unroll
            for (int hh = 1; hh < EPL; hh <<= 1)
#pragma unroll
                for (int r = 0; r < EPL; ++r)
                    if ((r & hh) == 0) {
                        const float u = a[r], w = a[r + hh];
                        a[r] = u + w;
                        a[r + hh] = u - w;
                    }
#pragma unroll
            for (int m = 1; m < 32; m <<= 1)
#pragma unroll
                for (int r = 0; r < EPL; ++r) {
                    const float o = __shfl_xor_sync(FULL, a[r], m);
                    a[r] = (lane & m) ? o - a[r] : a[r] + o;
                }
            const float rs = rsqrtf((float)D);
            __half* qt = reinterpret_cast<__half*>(smem + G::OFF_QT);
            __half* ql = reinterpret_cast<__half*>(smem + G::OFF_QL);
            __half* qf = reinterpret_cast<__half*>(smem + G::OFF_QF);
#pragma unroll
            for (int r = 0; r < EPL; ++r) {
                const int i = lane * EPL + r;
                {   // rotated query, natural slot order: block i/16, slot s = i%16
                    const int kb = i >> 4, s = i & 15;
                    const int at = (kb * 32 + 4 * hd + ((s & 7) >> 1)) * 4 + (s >> 3) * 2 + (s & 1);
                    // fp16 pair hi + lo carries the rotated query to ~2^-22
                    const float v = a[r] * rs;
                    const __half vh = __float2half_rn(v);
                    qt[at] = vh;
                    ql[at] = __float2half_rn(v - __half2float(vh));
                }
                {   // plain query in the slot order of the FP8 key loads: 16 consecutive dims per lane
                    const int j = i >> 6, t4 = (i & 63) >> 4, wv = (i & 15) >> 2, e = i & 3;
                    qf[((4 * j + wv) * 32 + 4 * hd + t4) * 4 + (e >> 1) * 2 + (e & 1)] = __float2half_rn(qx[r]);
                }
            }
        }
        __syncthreads();
        MKV_STAMP(2);

        {
            // With two warps per unit a slot is handed back one page late: the exchange barrier inside page
            // n+1 is what proves that both warps have finished reading page n.
            int id, index;
            bool pending = false;
            while (!failed && walker_next(cons, 1, id, index)) {
                wait_slot(tail);
                if (failed) break;
#ifdef MKV_EXP_NOCOMPUTE
                acc.l[0] += __uint_as_float(lds64(ring + tail * G::SLOT + lane * 8).x & 1u);
                if constexpr (HALVES == 2) unit_sync();
#else
                tq3_page<D, HALVES>(acc, ring + tail * G::SLOT, qt_lane, sc2, lane, px);
#endif
                tail = (tail + 1) & (NSTAGE - 1);
                if constexpr (HALVES == 2) {
                    if (pending) --in_flight;
                    pending = true;
                } else {
                    --in_flight;
                    __syncwarp();
                }
                produce_tq3();
            }
            if constexpr (HALVES == 2) {
                unit_sync();                  // both warps are done with the last page
                if (pending) --in_flight;
            }
        }

        // ---- pass over the Recent/Anchor (FP8) pages: two slots per page (keys, values) -------------
        if (n_my > 0 && !failed) {
            prod.chunk = 0;
            walker_load(prod, 0);
            cons = prod;
            prod_more = true;
            head = tail = 0;          // the ring is empty here; pairs sit at even positions
            auto produce_fp8 = [&]() {
                while (prod_more && !failed && in_flight + 2 <= NSTAGE) {
                    int id, index;
                    prod_more = walker_next(prod, 0, id, index);
                    if (!prod_more) break;
                    if (issuer) {
                        const uint8_t* rec = P.fp8 + ((size_t)id * hkv + h) * (2 * G::FP8_HALF);
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        mbar_expect_tx(bars + 8 * head, G::FP8_HALF);
                        bulk_load(ring + head * G::SLOT, rec, G::FP8_HALF, bars + 8 * head);
                        mbar_expect_tx(bars + 8 * (head + 1), G::FP8_HALF);
                        bulk_load(ring + (head + 1) * G::SLOT, rec + G::FP8_HALF, G::FP8_HALF, bars + 8 * (head + 1));
                    }
                    head = (head + 2) & (NSTAGE - 1);
                    in_flight += 2;
                }
            };
            produce_fp8();
            int id, index;
            bool pending = false;
            while (!failed && walker_next(cons, 0, id, index)) {
                wait_slot(tail);
                wait_slot(tail + 1);
                if (failed) break;
                const int pg = page_at(unit + NU * index);
                fp8_page<D, HALVES>(acc, ring + tail * G::SLOT, ring + (tail + 1) * G::SLOT, qf_lane, sc2 * P.k_scale,
                                    P.v_scale, min(kPage, len - pg * kPage), lane, px);
                tail = (tail + 2) & (NSTAGE - 1);
                if constexpr (HALVES == 2) {
                    if (pending) in_flight -= 2;
                    pending = true;
                } else {
                    in_flight -= 2;
                    __syncwarp();
                }
                produce_fp8();
            }
            if constexpr (HALVES == 2) {
                unit_sync();
                if (pending) in_flight -= 2;
            }
        }
        float (&oacc)[NBH][4] = acc.o;
        float (&lacc)[2] = acc.l;
        float (&m_run)[2] = acc.m;

        // ---- combine the warps of the block (ring memory is idle now) ---------------------------
        MKV_STAMP(3);
        __syncthreads();
        MKV_STAMP(4);
        if (g == 0 && hf == 0) {           // both warps of a unit hold the same maximum and row sums
            sm_m[unit * 8 + 2 * tq] = m_run[0];
            sm_m[unit * 8 + 2 * tq + 1] = m_run[1];
        }
        __syncthreads();
        float M0 = -CUDART_INF_F, M1 = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < NU; ++w) {
            M0 = fmaxf(M0, sm_m[w * 8 + 2 * tq]);
            M1 = fmaxf(M1, sm_m[w * 8 + 2 * tq + 1]);
        }
        {
            const float f0 = m_run[0] == -CUDART_INF_F ? 0.f : fast_exp2(m_run[0] - M0);
            const float f1 = m_run[1] == -CUDART_INF_F ? 0.f : fast_exp2(m_run[1] - M1);
            float* mine = red + (size_t)unit * D * 8 + (size_t)hf * NBH * 16 * 8;   // this warp's channel blocks
#pragma unroll
            for (int i = 0; i < NBH; ++i) {
                // element (channel 16i + g + 8*(e>>1), head 2tq + (e&1)) at [channel][8 heads]
                *reinterpret_cast<float2*>(mine + (16 * i + g) * 8 + 2 * tq) = make_float2(oacc[i][0] * f0, oacc[i][1] * f1);
                *reinterpret_cast<float2*>(mine + (16 * i + g + 8) * 8 + 2 * tq) = make_float2(oacc[i][2] * f0, oacc[i][3] * f1);
            }
            if (g == 0 && hf == 0) {
                sm_l[unit * 8 + 2 * tq] = lacc[0] * f0;
                sm_l[unit * 8 + 2 * tq + 1] = lacc[1] * f1;
            }
        }
        __syncthreads();

        MKV_STAMP(5);
        const bool whole_row = (pos == row_start) && (pos + n_seg == row_end);
        const int pair = b * hkv + h;
        if (whole_row) {
            for (int e = tid; e < 8 * D; e += NW * 32) {
                const int head = e & 7, ch = e >> 3;
                if (head >= GQ) continue;
                float acc = 0.f, l = 0.f;
#pragma unroll
                for (int w = 0; w < NU; ++w) {
                    acc += red[(size_t)w * D * 8 + e];
                    l += sm_l[w * 8 + head];
                }
                P.out[((size_t)b * hq + h * GQ + head) * D + ch] = l > 0.f ? acc / l : 0.f;
            }
            if (P.lse && tid < GQ) {
                float l = 0.f, M = -CUDART_INF_F;
                for (int w = 0; w < NU; ++w) {
                    l += sm_l[w * 8 + tid];
                    M = fmaxf(M, sm_m[w * 8 + tid]);
                }
                P.lse[(size_t)b * hq + h * GQ + tid] = l > 0.f ? (M + log2f(l)) * kLn2 : -CUDART_INF_F;
            }
        } else {
            // partial (m, l, O) of this block for the row; slot 2c if the segment opens the block's range
            float* slot = P.partials + (size_t)(2 * blockIdx.x + (pos != my_start ? 1 : 0)) * (8 * D + 16);
            for (int e = tid; e < 8 * D; e += NW * 32) {
                float acc = 0.f;
#pragma unroll
                for (int w = 0; w < NU; ++w) acc += red[(size_t)w * D * 8 + e];
                slot[e] = acc;
            }
            if (tid < 8) {
                float l = 0.f, M = -CUDART_INF_F;
                for (int w = 0; w < NU; ++w) {
                    l += sm_l[w * 8 + tid];
                    M = fmaxf(M, sm_m[w * 8 + tid]);
                }
                slot[8 * D + tid] = M;
                slot[8 * D + 8 + tid] = l;
            }
            __threadfence();
            __syncthreads();
            MKV_STAMP(6);
            const int c0 = block_of(row_start), c1 = block_of(row_end - 1);
            if (tid == 0) {
                const uint32_t t = atomicAdd(&P.tickets[pair], 1u);
                *sm_flag = (t == (uint32_t)(c1 - c0)) ? 1 : 0;
            }
            __syncthreads();
            MKV_STAMP(7);
            if (*sm_flag) {
                // last block of the row: Eq. (softmax-merge) over the row's partials
                __threadfence();
                const int n_parts = c1 - c0 + 1;
                int* pslot = reinterpret_cast<int*>(red);                 // [n_parts] slot index of each part
                float* pm = red + kMaxCtas;                               // [n_parts][8] partial maxima
                float* wts = pm + kMaxCtas * 8;                           // [n_parts][8] weights, then l
                for (int c = tid; c < n_parts; c += NW * 32)
                    pslot[c] = 2 * (c0 + c) + (row_start > range_start(c0 + c) ? 1 : 0);
                __syncthreads();
                for (int i = tid; i < n_parts * 8; i += NW * 32) {
                    const float* ps = P.partials + (size_t)pslot[i >> 3] * (8 * D + 16) + 8 * D;
                    const float lj = __ldcg(ps + 8 + (i & 7));
                    pm[i] = lj > 0.f ? __ldcg(ps + (i & 7)) : -CUDART_INF_F;
                    wts[i] = lj;
                }
                __syncthreads();
                if (tid < 8) {
                    float M = -CUDART_INF_F;
                    for (int c = 0; c < n_parts; ++c) M = fmaxf(M, pm[c * 8 + tid]);
                    sm_m[tid] = M;
                }
                __syncthreads();
                for (int i = tid; i < n_parts * 8; i += NW * 32) {
                    const float mj = pm[i];
                    wts[i] = mj == -CUDART_INF_F ? 0.f : fast_exp2(mj - sm_m[i & 7]) * wts[i];   // w_j * l_j
                    pm[i] = mj == -CUDART_INF_F ? 0.f : fast_exp2(mj - sm_m[i & 7]);              // w_j
                }
                __syncthreads();
                if (tid < 8) {
                    float L = 0.f;
                    for (int c = 0; c < n_parts; ++c) L += wts[c * 8 + tid];
                    sm_l[tid] = L;
                }
                __syncthreads();
                // four consecutive heads of one channel per thread; the loads of 16 partials are issued
                // together before any of them is used
                for (int e4 = tid; e4 < 2 * D; e4 += NW * 32) {
                    const int head0 = (e4 & 1) * 4, ch = e4 >> 1;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int c0b = 0; c0b < n_parts; c0b += 16) {
                        float4 v[16];
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            const int c = min(c0b + k, n_parts - 1);
                            v[k] = __ldcg(reinterpret_cast<const float4*>(P.partials + (size_t)pslot[c] * (8 * D + 16)) + e4);
                        }
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            if (c0b + k < n_parts) {
                                const float4 w = *reinterpret_cast<const float4*>(pm + (c0b + k) * 8 + head0);
                                acc.x = fmaf(w.x, v[k].x, acc.x);
                                acc.y = fmaf(w.y, v[k].y, acc.y);
                                acc.z = fmaf(w.z, v[k].z, acc.z);
                                acc.w = fmaf(w.w, v[k].w, acc.w);
                            }
                        }
                    }
                    const float av[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int head = head0 + k;
                        if (head < GQ) {
                            const float L = sm_l[head];
                            P.out[((size_t)b * hq + h * GQ + head) * D + ch] = L > 0.f ? av[k] / L : 0.f;
                        }
                    }
                }
                if (P.lse && tid < GQ)
                    P.lse[(size_t)b * hq + h * GQ + tid] = sm_l[tid] > 0.f ? (sm_m[tid] + log2f(sm_l[tid])) * kLn2 : -CUDART_INF_F;
                if (tid == 0) P.tickets[pair] = 0;         // leave the header clean for the next call
            }
        }
        __syncthreads();
        MKV_STAMP(8);
        pos += n_seg;
    }
}

template <int D, int NW, int NSTAGE, int MINB, int HALVES>
static int32_t run_tensor(mkv_pool* p, DecodeParams& prm, cudaStream_t s)
{
    using G = Geo<D, NW, NSTAGE, HALVES>;
    auto kern = decode_tensor_kernel<D, NW, NSTAGE, MINB, HALVES>;
    static int grid_cache[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int dev = p->device & 7;
    if (grid_cache[dev] == 0) {
        MKV_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM));
        int per_sm = 0;
        MKV_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, NW * 32, G::SMEM));
        if (per_sm < 1) return MKV_E_INVALID;
        int grid = p->dev.sm_count * per_sm;
        grid_cache[dev] = grid > kMaxCtas ? kMaxCtas : grid;
    }
    kern<<<grid_cache[dev], NW * 32, G::SMEM, s>>>(prm);
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
}

// launch shape: warps per block, ring slots per warp, blocks per SM the register budget is sized for
static int tensor_shape()
{
    static int shape = -1;
    if (shape < 0) {
        const char* e = getenv("MKV_DECODE_SHAPE");
        shape = e ? atoi(e) : 0;
    }
    return shape;
}

#ifdef MKV_TIMELINE
extern "C" int mkv_debug_timeline(unsigned long long* host, int n)
{
    return (int)cudaMemcpyFromSymbol(host, g_timeline, sizeof(unsigned long long) * n);
}
#endif

int32_t launch_decode_tensor(mkv_pool* p, const void* q, const int32_t* bt, const uint8_t* tags,
                             const int32_t* lens, int B, int max_pages, float scale, float* out, float* lse,
                             void* ws, size_t, cudaStream_t s)
{
    if (B > kMaxBatch) return MKV_E_INVALID;
    DecodeParams prm;
    prm.fp8 = p->fp8; prm.tq3 = p->tq3;
    prm.fp8_pages = p->cfg.fp8_pages; prm.tq3_pages = p->cfg.tq3_pages;
    prm.hkv = p->hkv; prm.group = p->group;
    prm.k_scale = p->cfg.k_scale; prm.v_scale = p->cfg.v_scale;
    prm.sigma = p->sigma;
    prm.q = static_cast<const __nv_bfloat16*>(q);
    prm.bt = bt; prm.tags = tags; prm.lens = lens;
    prm.B = B; prm.max_pages = max_pages; prm.scale = scale;
    prm.out = out; prm.lse = lse;
    prm.tickets = reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(ws) + 256);
    prm.partials = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + decode_ws_header_bytes(B, p->hkv));
    prm.status = p->status_dev;
    // Launch shapes, measured on B200 (2 x 59,008 tokens, d = 256): 8 warps with 255 registers and whole-page
    // warps stream as fast as 16 warps in pairs; MKV_DECODE_SHAPE selects the alternatives for profiling.
    const int shape = tensor_shape();
    if (p->d == 128) {
        switch (shape) {
        case 1: return run_tensor<128, 8, 4, 1, 1>(p, prm, s);
        case 2: return run_tensor<128, 12, 4, 1, 1>(p, prm, s);
        case 3: return run_tensor<128, 8, 2, 2, 1>(p, prm, s);
        default: return run_tensor<128, 16, 4, 1, 1>(p, prm, s);
        }
    }
    switch (shape) {
    case 1: return run_tensor<256, 16, 4, 1, 2>(p, prm, s);
    case 2: return run_tensor<256, 12, 4, 1, 1>(p, prm, s);
    case 3: return run_tensor<256, 8, 4, 2, 2>(p, prm, s);
    default: return run_tensor<256, 8, 4, 1, 1>(p, prm, s);
    }
}

}  // namespace mkv
