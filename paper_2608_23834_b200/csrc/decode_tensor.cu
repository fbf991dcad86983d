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

__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// same product with a zero accumulator: d = A B
__device__ __forceinline__ void mma16816_zero(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x)
{
    uint32_t r;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(r) : "r"(x));
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
    const uint32_t u = (x & mask) | 0x64006400u;
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
template <int D, int NW, int NSTAGE>
struct Geo {
    static constexpr int NB = D / 16;                       // 16-wide blocks along d
    static constexpr int LW = 3 * NB / 4;                   // packed words per lane and code section
    static constexpr int TQ3_REC = 16 * D + 32;
    static constexpr int FP8_HALF = 16 * D;
    static constexpr int SLOT = (TQ3_REC + 127) / 128 * 128;
    static constexpr int RING = NW * NSTAGE * SLOT;
    static constexpr int QFRAG = NB * 32 * 8;               // one set of query B fragments
    static constexpr int OFF_QT = RING;
    static constexpr int OFF_QL = OFF_QT + QFRAG;            // low-order halves of the rotated query
    static constexpr int OFF_QF = OFF_QL + QFRAG;
    static constexpr int OFF_BAR = OFF_QF + QFRAG;
    static constexpr int OFF_CUM = OFF_BAR + NW * NSTAGE * 8;
    static constexpr int OFF_M = OFF_CUM + (kMaxBatch + 1) * 4;
    static constexpr int OFF_L = OFF_M + NW * 8 * 4;
    static constexpr int OFF_FLAG = OFF_L + NW * 8 * 4;
    static constexpr int SMEM = OFF_FLAG + 16;
    static_assert(NSTAGE >= 2, "an FP8 page takes two slots");
    static_assert(NSTAGE * SLOT >= 8 * D * 4, "ring doubles as the cross-warp reduction buffer");
    static_assert(FP8_HALF <= SLOT, "half an FP8 record fits a slot");
    static_assert(RING >= kMaxCtas * 4 + 2 * kMaxCtas * 8 * 4, "ring doubles as the final-merge scratch");
};

#ifdef MKV_TIMELINE
__device__ unsigned long long g_timeline[kMaxCtas * 16];
#define MKV_STAMP(k)                                                                     \
    do {                                                                                 \
        if (threadIdx.x == 0 && tl_seg == 0) {                                            \
            unsigned long long t__;                                                      \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t__));                       \
            g_timeline[blockIdx.x * 16 + (k)] = t__;                                      \
        }                                                                                \
    } while (0)
#else
#define MKV_STAMP(k)
#endif

template <int D, int NW, int NSTAGE, int MINB>
__global__ void __launch_bounds__(NW * 32, MINB) decode_tensor_kernel(const DecodeParams P)
{
#ifdef MKV_TIMELINE
    int tl_seg = 0;
#endif
    MKV_STAMP(0);
    using G = Geo<D, NW, NSTAGE>;
    constexpr int NB = G::NB;
    constexpr uint32_t FULL = 0xffffffffu;
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    int* cum = reinterpret_cast<int*>(smem + G::OFF_CUM);
    float* sm_m = reinterpret_cast<float*>(smem + G::OFF_M);
    float* sm_l = reinterpret_cast<float*>(smem + G::OFF_L);
    int* sm_flag = reinterpret_cast<int*>(smem + G::OFF_FLAG);
    float* red = reinterpret_cast<float*>(smem);            // [NW][D][8] over the ring, between segments

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    const int hkv = P.hkv, GQ = P.group, hq = hkv * GQ;

    // ---- prologue: barriers, zero rows of empty requests, prefix of pages -----------------------
    if (tid == 0) {
        for (int i = 0; i < NW * NSTAGE; ++i) mbar_init(sbase + G::OFF_BAR + 8 * i, 1);
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

    // per-warp pipeline state (absolute slot counters keep the mbarrier phases consistent)
    uint32_t slot_head = 0, slot_tail = 0;
    bool failed = false;
    const uint32_t ring = sbase + warp * NSTAGE * G::SLOT;
    const uint32_t bars = sbase + G::OFF_BAR + warp * NSTAGE * 8;
    const float sc2 = P.scale * kLog2e;      // scores are kept in log2 units

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

        // ---- query fragments: one warp per head ------------------------------------------------
        for (int hd = warp; hd < 8; hd += NW) {
            constexpr int EPL = D / 32;
            float x[EPL], a[EPL];
#pragma unroll
            for (int r = 0; r < EPL; ++r) {
                const int i = lane * EPL + r;
                x[r] = hd < GQ ? __bfloat162float(P.q[((size_t)b * hq + h * GQ + hd) * D + i]) : 0.f;
                a[r] = ((P.sigma.w[i >> 5] >> (i & 31)) & 1u) ? -x[r] : x[r];
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
                    qf[((4 * j + wv) * 32 + 4 * hd + t4) * 4 + (e >> 1) * 2 + (e & 1)] = __float2half_rn(x[r]);
                }
            }
        }
        __syncthreads();
        MKV_STAMP(2);

        // ---- this warp's pages of the segment --------------------------------------------------
        const int n_my = warp < n_seg ? (n_seg - warp + NW - 1) / NW : 0;
        float oacc[NB][4];
#pragma unroll
        for (int i = 0; i < NB; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
        float lacc[2] = {0.f, 0.f};
        float m_run[2] = {-CUDART_INF_F, -CUDART_INF_F};

        // table entries of the warp's pages, 32 at a time (entry i of the chunk lives in lane i)
        int cur_id = 0, cur_tag = 0, nxt_id = 0, nxt_tag = 0;
        auto load_chunk = [&](int chunk, int& id, int& tag) {
            const int i = chunk * 32 + lane;
            id = 0;
            tag = 0;
            if (i < n_my) {
                const int pg = pg0 + warp + NW * i;
                id = bt_row[pg];
                tag = tag_row[pg];
            }
        };
        load_chunk(0, cur_id, cur_tag);
        load_chunk(1, nxt_id, nxt_tag);
        int cons_chunk = 0;
        // entry(i): id, tag and validity of the warp's i-th page (i within the current or next chunk)
        auto entry = [&](int i, int& id, int& tag, int& valid, bool& ok) {
            const bool in_cur = (i >> 5) == cons_chunk;
            id = __shfl_sync(FULL, in_cur ? cur_id : nxt_id, i & 31);
            tag = __shfl_sync(FULL, in_cur ? cur_tag : nxt_tag, i & 31);
            const int pg = pg0 + warp + NW * i;
            valid = min(kPage, len - pg * kPage);
            ok = tag == MKV_TAG_STALE ? (id >= 0 && id < P.tq3_pages && valid == kPage)
                                      : (tag <= MKV_TAG_ANCHOR && id >= 0 && id < P.fp8_pages);
        };
        int i_prod = 0;
        auto produce = [&]() {
            while (i_prod < n_my && !failed) {
                int id, tag, valid;
                bool ok;
                entry(i_prod, id, tag, valid, ok);
                if (ok) {
                    const uint32_t need = tag == MKV_TAG_STALE ? 1u : 2u;
                    if (NSTAGE - (slot_head - slot_tail) < need) break;
                    if (lane == 0) {
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        if (tag == MKV_TAG_STALE) {
                            const uint32_t s = slot_head % NSTAGE;
                            mbar_expect_tx(bars + 8 * s, G::TQ3_REC);
                            bulk_load(ring + s * G::SLOT, P.tq3 + ((size_t)id * hkv + h) * G::TQ3_REC, G::TQ3_REC, bars + 8 * s);
                        } else {
                            const uint8_t* rec = P.fp8 + ((size_t)id * hkv + h) * (2 * G::FP8_HALF);
                            const uint32_t s0 = slot_head % NSTAGE, s1 = (slot_head + 1) % NSTAGE;
                            mbar_expect_tx(bars + 8 * s0, G::FP8_HALF);
                            bulk_load(ring + s0 * G::SLOT, rec, G::FP8_HALF, bars + 8 * s0);
                            mbar_expect_tx(bars + 8 * s1, G::FP8_HALF);
                            bulk_load(ring + s1 * G::SLOT, rec + G::FP8_HALF, G::FP8_HALF, bars + 8 * s1);
                        }
                    }
                    slot_head += need;
                } else if (lane == 0) {
                    atomicOr(P.status, kStBounds);
                }
                ++i_prod;
            }
        };
        // bounded wait for the slot with absolute index s_abs
        auto wait_slot = [&](uint32_t s_abs) {
            const uint32_t bar = bars + 8 * (s_abs % NSTAGE), parity = (s_abs / NSTAGE) & 1u;
            bool done = false;
            for (int it = 0; it < (1 << 22) && !done; ++it) done = mbar_try_wait(bar, parity);
            if (!__all_sync(FULL, done)) {
                failed = true;
                if (lane == 0) atomicOr(P.status, kStTimeout);
            }
        };
        produce();

        for (int i_cons = 0; i_cons < n_my; ++i_cons) {
            if ((i_cons >> 5) != cons_chunk) {
                cons_chunk = i_cons >> 5;
                cur_id = nxt_id;
                cur_tag = nxt_tag;
                load_chunk(cons_chunk + 1, nxt_id, nxt_tag);
            }
            int id, tag, valid;
            bool ok;
            entry(i_cons, id, tag, valid, ok);
            if (!ok || failed) continue;
            const bool is_tq3 = tag == MKV_TAG_STALE;
            const uint32_t s_k = ring + (slot_tail % NSTAGE) * G::SLOT;
            const uint32_t s_v = is_tq3 ? s_k + 6 * D : ring + ((slot_tail + 1) % NSTAGE) * G::SLOT;
            wait_slot(slot_tail);
            if (failed) continue;

            // ================= S = K q^T : 16 tokens x 8 heads ===================================
            float S0[4] = {0.f, 0.f, 0.f, 0.f}, S1[4] = {0.f, 0.f, 0.f, 0.f};
            float row_scale0, row_scale1;          // per-token factor of rows g and g+8
            if (is_tq3) {
                const uint32_t qb = sbase + G::OFF_QT + lane * 8;
                uint32_t kw[G::LW];
#pragma unroll
                for (int c = 0; c < G::LW / 4; ++c) {
                    const uint4 v = lds128(s_k + c * 512 + lane * 16);
                    kw[4 * c] = v.x; kw[4 * c + 1] = v.y; kw[4 * c + 2] = v.z; kw[4 * c + 3] = v.w;
                }
                if (G::LW % 4) {
                    const uint2 v = lds64(s_k + (G::LW / 4) * 512 + lane * 8);
                    kw[G::LW - 2] = v.x; kw[G::LW - 1] = v.y;
                }
#pragma unroll
                for (int j = 0; j < NB / 4; ++j) {
                    const uint32_t A = kw[3 * j], Bw = kw[3 * j + 1], Cw = kw[3 * j + 2];
                    uint32_t sel[4];
                    sel[0] = A & 0x77777777u;
                    sel[1] = Bw & 0x77777777u;
                    sel[2] = (Cw & 0x33333333u) | ((A >> 1) & 0x44444444u);
                    sel[3] = ((Cw >> 2) & 0x33333333u) | ((Bw >> 1) & 0x44444444u);
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        uint32_t a[4];
                        key_lut4(sel[w], a[0], a[1]);
                        key_lut4(sel[w] >> 16, a[2], a[3]);
                        const uint2 qv = lds64(qb + (4 * j + w) * 256);
                        const uint2 qw = lds64(qb + G::QFRAG + (4 * j + w) * 256);
                        if (w & 1) { mma16816(S1, a, qv.x, qv.y); mma16816(S1, a, qw.x, qw.y); }
                        else       { mma16816(S0, a, qv.x, qv.y); mma16816(S0, a, qw.x, qw.y); }
                    }
                }
                const uint32_t gaddr = s_k + 12 * D;
                row_scale0 = __half2float(__ushort_as_half(lds16(gaddr + 2 * g))) * sc2;
                row_scale1 = __half2float(__ushort_as_half(lds16(gaddr + 2 * g + 16))) * sc2;
            } else {
                const uint32_t qb = sbase + G::OFF_QF + lane * 8;
#pragma unroll
                for (int j = 0; j < D / 64; ++j) {
                    const uint4 r0 = lds128(s_k + g * D + 64 * j + 16 * tq);
                    const uint4 r1 = lds128(s_k + (g + 8) * D + 64 * j + 16 * tq);
                    const uint32_t w0[4] = {r0.x, r0.y, r0.z, r0.w}, w1[4] = {r1.x, r1.y, r1.z, r1.w};
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        uint32_t a[4];
                        a[0] = e4m3x2_to_f16x2((uint16_t)(w0[w] & 0xFFFFu));
                        a[1] = e4m3x2_to_f16x2((uint16_t)(w1[w] & 0xFFFFu));
                        a[2] = e4m3x2_to_f16x2((uint16_t)(w0[w] >> 16));
                        a[3] = e4m3x2_to_f16x2((uint16_t)(w1[w] >> 16));
                        const uint2 qv = lds64(qb + (4 * j + w) * 256);
                        if (w & 1) mma16816(S1, a, qv.x, qv.y);
                        else       mma16816(S0, a, qv.x, qv.y);
                    }
                }
                row_scale0 = row_scale1 = sc2 * P.k_scale;
            }

            // ================= online softmax (log2 units), lazily raised maximum ================
            float s[4];
            s[0] = (S0[0] + S1[0]) * row_scale0;
            s[1] = (S0[1] + S1[1]) * row_scale0;
            s[2] = (S0[2] + S1[2]) * row_scale1;
            s[3] = (S0[3] + S1[3]) * row_scale1;
            if (valid < kPage) {
                if (g >= valid) s[0] = s[1] = -CUDART_INF_F;
                if (g + 8 >= valid) s[2] = s[3] = -CUDART_INF_F;
            }
            float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(FULL, mx0, o));
                mx1 = fmaxf(mx1, __shfl_xor_sync(FULL, mx1, o));
            }
            const bool up0 = mx0 > m_run[0] + kRescaleSlack, up1 = mx1 > m_run[1] + kRescaleSlack;
            if (__any_sync(FULL, up0 || up1)) {
                const float f0 = up0 ? fast_exp2(m_run[0] - mx0) : 1.f, f1 = up1 ? fast_exp2(m_run[1] - mx1) : 1.f;
                if (up0) m_run[0] = mx0;
                if (up1) m_run[1] = mx1;
#pragma unroll
                for (int i = 0; i < NB; ++i) {
                    oacc[i][0] *= f0; oacc[i][2] *= f0;
                    oacc[i][1] *= f1; oacc[i][3] *= f1;
                }
                lacc[0] *= f0;
                lacc[1] *= f1;
            }
            const float p0 = fast_exp2(s[0] - m_run[0]), p1 = fast_exp2(s[1] - m_run[1]);
            const float p2 = fast_exp2(s[2] - m_run[0]), p3 = fast_exp2(s[3] - m_run[1]);
            // P^T as the B operand (tokens along k, heads along n), as an fp16 pair hi + lo
            const uint32_t ph01 = pack_f16x2(p0, p1), ph23 = pack_f16x2(p2, p3);
            const float2 h01 = half2_to_float2(ph01), h23 = half2_to_float2(ph23);
            const uint32_t pb0 = movmatrix_trans(ph01), pb1 = movmatrix_trans(ph23);
            const uint32_t pc0 = movmatrix_trans(pack_f16x2(p0 - h01.x, p1 - h01.y));
            const uint32_t pc1 = movmatrix_trans(pack_f16x2(p2 - h23.x, p3 - h23.y));
            float ps[4];
            {   // row sums of this page through the tensor core (the same P as the PV product)
                const uint32_t ones[4] = {0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u};
                mma16816_zero(ps, ones, pb0, pb1);
                mma16816(ps, ones, pc0, pc1);
                lacc[0] += ps[0];
                lacc[1] += ps[1];
            }

            // ================= O^T += V^T P : d channels x 8 heads ================================
            if (is_tq3) {
                uint32_t vw[G::LW];
#pragma unroll
                for (int c = 0; c < G::LW / 4; ++c) {
                    const uint4 v = lds128(s_v + c * 512 + lane * 16);
                    vw[4 * c] = v.x; vw[4 * c + 1] = v.y; vw[4 * c + 2] = v.z; vw[4 * c + 3] = v.w;
                }
                if (G::LW % 4) {
                    const uint2 v = lds64(s_v + (G::LW / 4) * 512 + lane * 8);
                    vw[G::LW - 2] = v.x; vw[G::LW - 1] = v.y;
                }
                const uint32_t meta = s_k + 12 * D + 32 + g * 16;
#pragma unroll
                for (int j = 0; j < NB / 4; ++j) {
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
                        affine_accumulate(oacc[4 * j], t, mt.x, mt.y, ps[0], ps[1]);
                        a[0] = value_code<4>(X1);
                        a[1] = value_code<7>(X1);
                        a[2] = value_code<2>(W1);
                        a[3] = value_code<5>(W1);
                        mma16816_zero(t, a, pb0, pb1);
                        mma16816(t, a, pc0, pc1);
                        affine_accumulate(oacc[4 * j + 1], t, mt.z, mt.w, ps[0], ps[1]);
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
                        affine_accumulate(oacc[4 * j + 2], t, mt.x, mt.y, ps[0], ps[1]);
                        a[0] = value_code<4>(W2);
                        a[1] = value_code<7>(W2);
                        a[2] = value_code<2>(X2);
                        a[3] = value_code<5>(X2);
                        mma16816_zero(t, a, pb0, pb1);
                        mma16816(t, a, pc0, pc1);
                        affine_accumulate(oacc[4 * j + 3], t, mt.z, mt.w, ps[0], ps[1]);
                    }
                }
                slot_tail += 1;
            } else {
                wait_slot(slot_tail + 1);
                if (failed) continue;
                const float vsc = P.v_scale;
                const bool scale_v = vsc != 1.0f;
                // bytes of tokens beyond the sequence end are cleared so that stale NaN patterns cannot leak
                uint32_t keep_lo = 0xFFFFu, keep_hi = 0xFFFFu;   // byte masks for tokens (2tq,2tq+1), (2tq+8,2tq+9)
                if (valid < kPage) {
                    keep_lo = (2 * tq < valid ? 0x00FFu : 0u) | (2 * tq + 1 < valid ? 0xFF00u : 0u);
                    keep_hi = (2 * tq + 8 < valid ? 0x00FFu : 0u) | (2 * tq + 9 < valid ? 0xFF00u : 0u);
                }
#pragma unroll
                for (int cb = 0; cb < NB; ++cb) {
                    const uint32_t r0 = s_v + (16 * cb + g) * 16 + 2 * tq, r1 = r0 + 8 * 16;
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
                        for (int e = 0; e < 4; ++e) oacc[cb][e] = fmaf(vsc, t[e], oacc[cb][e]);
                    } else {
                        mma16816(oacc[cb], a, pb0, pb1);
                        mma16816(oacc[cb], a, pc0, pc1);
                    }
                }
                slot_tail += 2;
            }
            __syncwarp();
            produce();
        }

        // ---- combine the warps of the block (ring memory is idle now) ---------------------------
        MKV_STAMP(3);
        __syncthreads();
        MKV_STAMP(4);
        if (g == 0) {
            sm_m[warp * 8 + 2 * tq] = m_run[0];
            sm_m[warp * 8 + 2 * tq + 1] = m_run[1];
        }
        __syncthreads();
        float M0 = -CUDART_INF_F, M1 = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            M0 = fmaxf(M0, sm_m[w * 8 + 2 * tq]);
            M1 = fmaxf(M1, sm_m[w * 8 + 2 * tq + 1]);
        }
        {
            const float f0 = m_run[0] == -CUDART_INF_F ? 0.f : fast_exp2(m_run[0] - M0);
            const float f1 = m_run[1] == -CUDART_INF_F ? 0.f : fast_exp2(m_run[1] - M1);
            float* mine = red + (size_t)warp * D * 8;
#pragma unroll
            for (int i = 0; i < NB; ++i) {
                // element (channel 16i + g + 8*(e>>1), head 2tq + (e&1)) at [channel][8 heads]
                *reinterpret_cast<float2*>(mine + (16 * i + g) * 8 + 2 * tq) = make_float2(oacc[i][0] * f0, oacc[i][1] * f1);
                *reinterpret_cast<float2*>(mine + (16 * i + g + 8) * 8 + 2 * tq) = make_float2(oacc[i][2] * f0, oacc[i][3] * f1);
            }
            if (g == 0) {
                sm_l[warp * 8 + 2 * tq] = lacc[0] * f0;
                sm_l[warp * 8 + 2 * tq + 1] = lacc[1] * f1;
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
                for (int w = 0; w < NW; ++w) {
                    acc += red[(size_t)w * D * 8 + e];
                    l += sm_l[w * 8 + head];
                }
                P.out[((size_t)b * hq + h * GQ + head) * D + ch] = l > 0.f ? acc / l : 0.f;
            }
            if (P.lse && tid < GQ) {
                float l = 0.f, M = -CUDART_INF_F;
                for (int w = 0; w < NW; ++w) {
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
                for (int w = 0; w < NW; ++w) acc += red[(size_t)w * D * 8 + e];
                slot[e] = acc;
            }
            if (tid < 8) {
                float l = 0.f, M = -CUDART_INF_F;
                for (int w = 0; w < NW; ++w) {
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
                // four consecutive heads of one channel per thread; many independent loads in flight
                for (int e4 = tid; e4 < 2 * D; e4 += NW * 32) {
                    const int head0 = (e4 & 1) * 4, ch = e4 >> 1;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
                    for (int c = 0; c < n_parts; ++c) {
                        const float4 v = __ldcg(reinterpret_cast<const float4*>(P.partials + (size_t)pslot[c] * (8 * D + 16)) + e4);
                        const float4 w = *reinterpret_cast<const float4*>(pm + c * 8 + head0);
                        acc.x = fmaf(w.x, v.x, acc.x);
                        acc.y = fmaf(w.y, v.y, acc.y);
                        acc.z = fmaf(w.z, v.z, acc.z);
                        acc.w = fmaf(w.w, v.w, acc.w);
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
#ifdef MKV_TIMELINE
        ++tl_seg;
#endif
        pos += n_seg;
    }
}

template <int D, int NW, int NSTAGE, int MINB>
static int32_t run_tensor(mkv_pool* p, DecodeParams& prm, cudaStream_t s)
{
    using G = Geo<D, NW, NSTAGE>;
    auto kern = decode_tensor_kernel<D, NW, NSTAGE, MINB>;
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
    const int shape = tensor_shape();
    if (p->d == 128) {
        switch (shape) {
        case 1: return run_tensor<128, 8, 2, 2>(p, prm, s);
        case 2: return run_tensor<128, 12, 3, 1>(p, prm, s);
        case 3: return run_tensor<128, 16, 2, 1>(p, prm, s);
        case 4: return run_tensor<128, 8, 3, 3>(p, prm, s);
        default: return run_tensor<128, 8, 3, 1>(p, prm, s);
        }
    }
    switch (shape) {
    case 1: return run_tensor<256, 8, 2, 2>(p, prm, s);
    case 2: return run_tensor<256, 12, 3, 1>(p, prm, s);
    case 3: return run_tensor<256, 16, 2, 1>(p, prm, s);
    case 4: return run_tensor<256, 4, 3, 3>(p, prm, s);
    default: return run_tensor<256, 8, 3, 1>(p, prm, s);
    }
}

}  // namespace mkv
