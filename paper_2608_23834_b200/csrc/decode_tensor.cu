// Tensor-core decode attention (MKV_DECODE_TENSOR): one-pass mixed-format split-KV scan.
//
// Section 3.3 / 4.1: every page of a request row is read in its own physical format (FP8 for
// Recent/Anchor, TQ3 for Stale), all tokens share one softmax, the whole GQA group reuses each
// unpacked tile, and split partials (m, l, O) are merged with Eq. (softmax-merge).
//
// Mapping to the hardware
//   * work = (request, KV head, page) triples in row-major order, cut into equal contiguous ranges,
//     one per block (persistent grid, a multiple of the SM count); a block processes the
//     (request, KV head) segments of its range one after another, its warps taking contiguous runs of pages.
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
//     workspace; every such block then takes a ticket of its row, and the block that draws the last
//     ticket combines the row's partials (Eq. softmax-merge) and writes the output.  No block ever
//     waits for another, and there is no second launch.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <math_constants.h>

#include <cstdlib>
#include <mutex>

#include "mkv_internal.cuh"

namespace mkv {

constexpr int kMaxBatch = 1024;      // requests per call
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleSlack = 8.0f;   // running maximum is only raised when exceeded by 2^8
constexpr unsigned long long kDefaultWaitNs = 20000000ull;   // 20 ms: far beyond any copy that is going to arrive

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
    int tiles;             // 16-token tiles per page (page = 16 * tiles tokens); table entries are per page
    float scale;
    float* out;
    float* lse;
    float* partials;       // [2 * grid][8*D + 16]
    uint32_t* tickets;     // [max_blocks] arrival counters of split rows, indexed by the row's first block; zero between calls
    int max_blocks;        // the partial area holds 2 * max_blocks slots
    float* mass;           // scored variant: [B][hq][max_pages], log2-domain page sums from the scan (else unused)
    uint32_t* status;
    unsigned long long wait_ns;   // wall-time limit of a wait for a page copy (kDefaultWaitNs unless the pool says otherwise)
};

// One launch can scan the pools of several layers (Section 4.1 runs the decode step of all full-attention
// layers from one CUDA graph): the layers share the requests (lengths, batch, geometry) and differ in
// their arenas, tables, queries, outputs and workspaces.  A block walks its share of layer 0, then of
// layer 1, ... without waiting for the other blocks, so the start-up and the merge tail of one layer
// overlap the page loops of its neighbours.
constexpr int kMaxLayers = 32;
template <int MAXL>
struct LayerSet {
    int n;
    DecodeParams layer[MAXL];
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

// D += A B with signed 8-bit integer operands and 32-bit integer accumulators: A 16 x 32 (row-major fragment),
// B 32 x 8.  (Measured on B200: this legacy integer MMA is one native instruction at the rate of the fp16
// m16n8k16 one, i.e. twice its products per instruction; the e4m3 form of mma.sync is expanded by the compiler
// into conversions and fp16 MMAs and is slower than the fp16 path it was meant to replace.)
__device__ __forceinline__ void mma16832_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// the same product with a zero accumulator
__device__ __forceinline__ void mma16832_s8_zero(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
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

__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
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
// The multiplier of the value unpack is read from the constant bank.  Written as a literal it needs a register
// (the inline PTX takes register operands) beside the one of the addend, and the scan is short of registers: the
// compiler then rebuilds literals with a move before every use.  Measured: 2 % of a layer's time; doing the same
// to the masks of the LOP3s, or writing these operations as plain expressions, made the scan slower.
// 2^-POS as fp16 pairs (exponent arithmetic on 1.0 = 0x3C00)
__constant__ uint32_t kValueMul[8] = {0x3C003C00u, 0x38003800u, 0x34003400u, 0x30003000u,
                                      0x2C002C00u, 0x28002800u, 0x24002400u, 0x20002000u};
template <int POS, bool CB = false>      // CB: multiplier from the constant bank (it pays in the format-2 scan only)
__device__ __forceinline__ uint32_t value_code(uint32_t x)
{
    constexpr uint32_t mask = 0x00070007u << POS;
    const uint32_t u = lop3_and_or(x, mask, 0x64006400u);
    // 2^-POS and -1024 * 2^-POS as fp16 pairs (exponent arithmetic on 1.0 = 0x3C00, -1024 = 0xE400)
    constexpr uint32_t mul = (0x3C00u - (POS << 10)) * 0x00010001u;
    constexpr uint32_t add = (0xE400u - (POS << 10)) * 0x00010001u;
    return hfma2_u32(u, CB ? kValueMul[POS] : mul, add);
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
// Work partition (the scan and the merge of split rows use the same cut)
// ------------------------------------------------------------------------------------------------
// Work = (request, KV head, page) triples in row-major order; cum[b] = index of the first triple of
// request b.  Two ways to cut it into one contiguous range per block:
//   row-aligned (few rows: B * hkv <= grid / 4): every row gets a whole number of blocks in proportion
//     to its pages (cumulative rounding), so that no block straddles two rows and pays the per-row set-up
//     and reduction twice;
//   linear (many rows): grid equal ranges that may cross row boundaries.
constexpr int kMaxAlignedRows = kMaxCtas / 4;

struct Partition {
    int aligned;                        // 1: row-aligned, 0: linear
    int blocks;                         // blocks that get work
    int base[kMaxAlignedRows + 1];      // row-aligned: first block of every row
};

// Called by warp 0 (all 32 lanes) after cum[] is complete; other warps wait at the next barrier.
__device__ __forceinline__ void build_partition(Partition* pt, const int* cum, int B, int hkv, int grid, int lane)
{
    constexpr uint32_t FULL = 0xffffffffu;
    const long long W = cum[B];
    const int rows = B * hkv;
    int blocks = (int)(W < (long long)grid ? W : (long long)grid);
    // With k blocks per row the rows that get one block fewer run 1/k longer, but a block that straddles two rows
    // pays the per-row set-up, reduction and partial twice (about 8 us, a quarter of a block's pages at config-1
    // sizes).  Measured: from four blocks per row on, whole blocks per row win (16 rows: 71 -> 66 us, 32 rows: 74 -> 71).
    int aligned = (rows * 4 <= grid && rows <= kMaxAlignedRows && W >= grid) ? 1 : 0;
    if (aligned) {
        // block boundaries at the rounded cumulative share of the rows: base[r] = round(grid * first_page(r) / W);
        // every row must end up with at least one block, otherwise the linear cut is used
        int bad = 0;
        const float scale = (float)grid / (float)W;
        for (int r = lane; r <= rows; r += 32) {
            int first = (int)W;                                 // r == rows: one past the last row
            if (r < rows) {
                const int b = r / hkv, h = r - b * hkv;
                first = cum[b] + h * ((cum[b + 1] - cum[b]) / hkv);
            }
            pt->base[r] = r == rows ? grid : (int)((float)first * scale + 0.5f);
        }
        __syncwarp();
        for (int r = lane; r < rows; r += 32) {
            const int b = r / hkv;
            if (cum[b + 1] > cum[b] && pt->base[r + 1] <= pt->base[r]) bad = 1;
        }
        if (__any_sync(FULL, bad)) aligned = 0;
        else blocks = grid;
    }
    if (lane == 0) {
        pt->aligned = aligned;
        pt->blocks = blocks;
    }
}

// linear range [start, end) of block c
__device__ __forceinline__ void partition_range(const Partition* pt, const int* cum, int hkv, int B, int c, int& start,
                                                int& end)
{
    const long long W = cum[B];
    if (!pt->aligned) {
        start = (int)((W * c) / pt->blocks);
        end = (int)((W * (c + 1)) / pt->blocks);
        return;
    }
    const int rows = B * hkv;
    int lo = 0;                                     // row of block c: base[r] <= c < base[r + 1]
    for (int hi = rows - 1; lo < hi;) {
        const int mid = (lo + hi) >> 1;
        if (pt->base[mid + 1] <= c) lo = mid + 1; else hi = mid;
    }
    const int r = lo, b = r / hkv, h = r - b * hkv, n = (cum[b + 1] - cum[b]) / hkv;
    const unsigned k = pt->base[r + 1] - pt->base[r], j = c - pt->base[r];
    const int row_start = cum[b] + h * n;
    start = row_start + (int)(((unsigned)n * j) / k);
    end = row_start + (int)(((unsigned)n * (j + 1)) / k);
}

__device__ __forceinline__ int partition_start(const Partition* pt, const int* cum, int hkv, int B, int c)
{
    int s, e;
    partition_range(pt, cum, hkv, B, c, s, e);
    return s;
}

// blocks c0..c1 that hold a part of the row [row_start, row_end) (row index r)
__device__ __forceinline__ void partition_blocks_of_row(const Partition* pt, const int* cum, int B, int r, int row_start,
                                                        int row_end, int& c0, int& c1)
{
    if (pt->aligned) {
        c0 = pt->base[r];
        c1 = pt->base[r + 1] - 1;
        return;
    }
    const long long W = cum[B];
    const int C = pt->blocks;
    auto start = [&](int c) -> int { return (int)((W * c) / C); };
    auto block_of = [&](int x) -> int {
        int c = (int)(((long long)x * C) / W);
        while (c + 1 < C && start(c + 1) <= x) ++c;
        while (c > 0 && start(c) > x) --c;
        return c;
    };
    c0 = block_of(row_start);
    c1 = block_of(row_end - 1);
}

// ------------------------------------------------------------------------------------------------
// kernel
// ------------------------------------------------------------------------------------------------

template <int D, int NW, int NSTAGE, bool SHORT_ROUNDS = false>
struct Geo {
    static constexpr int NB = D / 16;                       // 16-wide blocks along d
    static constexpr int LW = 3 * NB / 4;                   // packed words per lane and code section
    static constexpr int TQ3_REC = 16 * D + 32;
    static constexpr int FP8_HALF = 16 * D;
    static constexpr int SLOT = (TQ3_REC + 127) / 128 * 128;
    // pages of one warp whose table entries are compacted at a time (fewer where the ring leaves little room)
    static constexpr int ROUND = (NW * NSTAGE * SLOT > 190000 || SHORT_ROUNDS) ? 64 : 128;
    static constexpr int RING = NW * NSTAGE * SLOT;
    static constexpr int QROT = NB * 32 * 16;               // rotated query B fragments, hi and lo interleaved
    static constexpr int QPLAIN = NB * 32 * 8;              // plain query B fragments (FP8 pages)
    static constexpr int OFF_QT = RING;
    static constexpr int OFF_QF = OFF_QT + QROT;
    static constexpr int OFF_BAR = OFF_QF + QPLAIN;
    static constexpr int OFF_LIST = OFF_BAR + NW * NSTAGE * 8;   // [warp][2 formats][ROUND] page ids, then [warp][2][ROUND] logical pages
    static constexpr int OFF_CUM = OFF_LIST + NW * 4 * ROUND * 4;
    static constexpr int OFF_STRIDE = OFF_CUM + (kMaxBatch + 1) * 4;
    static constexpr int OFF_M = OFF_STRIDE + kMaxBatch * 4;
    static constexpr int OFF_L = OFF_M + NW * 8 * 4;
    static constexpr int OFF_PART = OFF_L + NW * 8 * 4;
    static constexpr int OFF_LAST = OFF_PART + ((int)sizeof(Partition) + 15) / 16 * 16;
    static constexpr int OFF_QS = OFF_LAST + 16;             // record format 2: digit unit of the rotated query, per head
    static constexpr int SMEM = OFF_QS + 32;
    static_assert(SLOT % 128 == 0 && OFF_QT % 16 == 0 && OFF_QF % 16 == 0 && OFF_BAR % 8 == 0,
                  "slots are bulk-copy destinations; query fragments are read with 16- and 8-byte loads");
    static_assert(NW >= 4, "a warp builds the query fragments of at most two columns of the 8-wide head group");
    static_assert(NSTAGE >= 2 && NSTAGE % 2 == 0 && NSTAGE <= 16, "an FP8 page takes a pair of slots; one phase bit per slot");
    static_assert(NSTAGE * SLOT >= 8 * D * 4, "ring doubles as the cross-warp reduction buffer");
    static_assert(FP8_HALF <= SLOT, "half an FP8 record fits a slot");
};


// Running state of one warp for one (request, KV head) segment: O^T accumulators [d channels x 8
// heads] in the MMA C layout, row sums and the (lazily raised) running maximum of the two head
// columns this lane owns, all in log2 units.
template <int NB>
struct WarpAcc {
    float o[NB][4];
    float l[2];
    float m[2];
    // pages of several tiles only: while the tiles of one Stale page are scanned, o holds sum p * code of
    // that page (the page's scale/zero are applied once, when the page is left), lp its row sums, and the
    // output accumulated before sits in shared memory, to be multiplied by pk (the rescales since then)
    float lp[2];
    float pk[2];
    // record format 2: its score tile has the heads in the rows, so the lane also keeps the running maximum
    // of head g (`mr`); m[] (heads 2tq, 2tq+1: the columns of the output tile) stays the master copy that the
    // Recent/Anchor pages, the page mass and the reduction use, and the two are brought in line on every change
    float mr;
};

// Scores of one page -> probabilities.  s[0..1] = token g, s[2..3] = token g+8 (heads 2tq, 2tq+1).
// Updates the running maximum (only when it is exceeded by more than 2^kRescaleSlack, so that
// accumulators are rarely rescaled), and returns P^T as MMA B fragments split into an fp16 pair
// hi (pb) + lo (pc), plus the page's row sums ps[0..1].
struct PFrag {
    uint32_t b0, b1, c0, c1;
    float ps0, ps1;
};

// First half: raise the running maximum (and rescale the accumulators) if the page asks for it.
template <int NB, bool TILED = false>
__device__ __forceinline__ void softmax_rescale(WarpAcc<NB>& acc, const float (&s)[4])
{
    constexpr uint32_t FULL = 0xffffffffu;
    float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
    // the page maximum is only needed when some score exceeds the running maximum by more than the slack
    if (__any_sync(FULL, mx0 > acc.m[0] + kRescaleSlack || mx1 > acc.m[1] + kRescaleSlack)) {
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
            mx0 = fmaxf(mx0, __shfl_xor_sync(FULL, mx0, o));
            mx1 = fmaxf(mx1, __shfl_xor_sync(FULL, mx1, o));
        }
        const bool up0 = mx0 > acc.m[0] + kRescaleSlack, up1 = mx1 > acc.m[1] + kRescaleSlack;
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
        if constexpr (TILED) {
            acc.lp[0] *= f0; acc.lp[1] *= f1;
            acc.pk[0] *= f0; acc.pk[1] *= f1;
        }
    }
}

// Second half, branch-free (so that it can be scheduled into the unpack work of the next page): P and its row sums.
template <int NB>
__device__ __forceinline__ void softmax_probs(WarpAcc<NB>& acc, const float (&s)[4], PFrag& pf)
{
    const float p0 = fast_exp2(s[0] - acc.m[0]), p1 = fast_exp2(s[1] - acc.m[1]);
    const float p2 = fast_exp2(s[2] - acc.m[0]), p3 = fast_exp2(s[3] - acc.m[1]);
    const uint32_t ph01 = pack_f16x2(p0, p1), ph23 = pack_f16x2(p2, p3);
    const float2 h01 = half2_to_float2(ph01), h23 = half2_to_float2(ph23);
    pf.b0 = movmatrix_trans(ph01);
    pf.b1 = movmatrix_trans(ph23);
    pf.c0 = movmatrix_trans(pack_f16x2(p0 - h01.x, p1 - h01.y));
    pf.c1 = movmatrix_trans(pack_f16x2(p2 - h23.x, p3 - h23.y));
    // row sums through the tensor core: the same P that multiplies V
    const uint32_t ones[4] = {0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u};
    float ps[4];
    mma16816_zero(ps, ones, pf.b0, pf.b1);
    mma16816(ps, ones, pf.c0, pf.c1);
    pf.ps0 = ps[0];
    pf.ps1 = ps[1];
    acc.l[0] += ps[0];
    acc.l[1] += ps[1];
}

template <int NB>
__device__ __forceinline__ void softmax_page(WarpAcc<NB>& acc, const float (&s)[4], PFrag& pf)
{
    softmax_rescale<NB>(acc, s);
    softmax_probs<NB>(acc, s, pf);
}

// Scored variant (Section 3.1): log2 of the page's exponential sum, referred to an absolute origin
// (row sum relative to the running maximum, plus that maximum), for the two heads this lane owns.
// mass_pg points at (request, first head of the group, this page); heads are mass_stride apart.
// The finishing kernel turns it into the globally normalised mass with the row's log-sum-exp.
// *addr <- log2(2^*addr + 2^v): several warps add their parts of one page's exponential sum (pages of several
// tiles); the entries start at -inf.
__device__ __forceinline__ void atomic_log2_add(float* addr, float v)
{
    int* ia = reinterpret_cast<int*>(addr);
    int old = *reinterpret_cast<volatile int*>(ia), assumed;
    do {
        assumed = old;
        const float a = __int_as_float(assumed);
        const float hi = fmaxf(a, v), lo = fminf(a, v);
        const float nv = lo == -CUDART_INF_F ? hi : hi + __log2f(1.f + fast_exp2(lo - hi));
        old = atomicCAS(ia, assumed, __float_as_int(nv));
    } while (old != assumed);
}

// ACCUMULATE: the entry receives a part of the page (a tile, or a run of tiles) and is added to, not stored.
template <int NB, bool ACCUMULATE = false>
__device__ __forceinline__ void store_page_mass(const WarpAcc<NB>& acc, float ps0, float ps1, float* mass_pg, int mass_stride,
                                                int GQ, int lane)
{
    if (lane < 4) {                  // g == 0: one lane per head pair
        const int h0 = 2 * lane;
        const float v0 = __log2f(ps0) + acc.m[0], v1 = __log2f(ps1) + acc.m[1];
        if constexpr (ACCUMULATE) {
            if (h0 < GQ) atomic_log2_add(mass_pg + (size_t)h0 * mass_stride, v0);
            if (h0 + 1 < GQ) atomic_log2_add(mass_pg + (size_t)(h0 + 1) * mass_stride, v1);
        } else {
            if (h0 < GQ) mass_pg[(size_t)h0 * mass_stride] = v0;
            if (h0 + 1 < GQ) mass_pg[(size_t)(h0 + 1) * mass_stride] = v1;
        }
    }
}

// All packed words of one lane for one code section.
template <int D>
__device__ __forceinline__ void load_lane_words(uint32_t sec, int lane, uint32_t (&w)[3 * (D / 16) / 4])
{
    constexpr int LW = 3 * (D / 16) / 4;
#pragma unroll
    for (int c = 0; c < LW / 4; ++c) {
        const uint4 v = lds128(sec + c * 512 + lane * 16);
        w[4 * c] = v.x; w[4 * c + 1] = v.y; w[4 * c + 2] = v.z; w[4 * c + 3] = v.w;
    }
    if constexpr (LW % 4 != 0) {
        const uint2 v = lds64(sec + (LW / 4) * 512 + lane * 8);
        w[LW - 2] = v.x; w[LW - 1] = v.y;
    }
}

// Scores of the four key blocks 4j..4j+3 of a Stale page: 12 byte-table lookups per block pair and two
// MMAs per block (query hi and lo).
__device__ __forceinline__ void tq3_key_quad(float (&S0)[4], float (&S1)[4], uint32_t A, uint32_t Bw, uint32_t Cw,
                                             uint32_t q_quad)
{
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
        const uint4 q = lds128(q_quad + w * 512);          // {hi b0, hi b1, lo b0, lo b1}
        if (w & 1) { mma16816(S1, a, q.x, q.y); mma16816(S1, a, q.z, q.w); }
        else       { mma16816(S0, a, q.x, q.y); mma16816(S0, a, q.z, q.w); }
    }
}

// Output update of the four channel blocks 4j..4j+3 of a Stale page: integer codes through the tensor
// core, then the fp16 scale and zero of every channel applied to the 16x8 result in fp32.
template <bool DEFER = false, bool CB = false>
__device__ __forceinline__ void tq3_value_quad(float (&o0)[4], float (&o1)[4], float (&o2)[4], float (&o3)[4],
                                               uint32_t W0, uint32_t W1, uint32_t W2, uint32_t meta_quad, const PFrag& pf)
{
    float t[4];
    uint32_t a[4];
    if constexpr (DEFER) {
        // sum p * code only: the accumulators are in code units until the page is left
        const uint32_t X1 = prmt(W0, W1, 0x6341u), X0 = prmt(W1, W2, 0x6341u), X2 = W2 >> 8;
        a[0] = value_code<0, CB>(W0); a[1] = value_code<3, CB>(W0); a[2] = value_code<6, CB>(W0); a[3] = value_code<1, CB>(X1);
        mma16816(o0, a, pf.b0, pf.b1);
        mma16816(o0, a, pf.c0, pf.c1);
        a[0] = value_code<4, CB>(X1); a[1] = value_code<7, CB>(X1); a[2] = value_code<2, CB>(W1); a[3] = value_code<5, CB>(W1);
        mma16816(o1, a, pf.b0, pf.b1);
        mma16816(o1, a, pf.c0, pf.c1);
        a[0] = value_code<0, CB>(X0); a[1] = value_code<3, CB>(X0); a[2] = value_code<6, CB>(X0); a[3] = value_code<1, CB>(W2);
        mma16816(o2, a, pf.b0, pf.b1);
        mma16816(o2, a, pf.c0, pf.c1);
        a[0] = value_code<4, CB>(W2); a[1] = value_code<7, CB>(W2); a[2] = value_code<2, CB>(X2); a[3] = value_code<5, CB>(X2);
        mma16816(o3, a, pf.b0, pf.b1);
        mma16816(o3, a, pf.c0, pf.c1);
        return;
    }
    {   // blocks 4j, 4j+1
        const uint4 mt = lds128(meta_quad);
        const uint32_t X1 = prmt(W0, W1, 0x6341u);
        a[0] = value_code<0, CB>(W0);
        a[1] = value_code<3, CB>(W0);
        a[2] = value_code<6, CB>(W0);
        a[3] = value_code<1, CB>(X1);
        mma16816_zero(t, a, pf.b0, pf.b1);
        mma16816(t, a, pf.c0, pf.c1);
        affine_accumulate(o0, t, mt.x, mt.y, pf.ps0, pf.ps1);
        a[0] = value_code<4, CB>(X1);
        a[1] = value_code<7, CB>(X1);
        a[2] = value_code<2, CB>(W1);
        a[3] = value_code<5, CB>(W1);
        mma16816_zero(t, a, pf.b0, pf.b1);
        mma16816(t, a, pf.c0, pf.c1);
        affine_accumulate(o1, t, mt.z, mt.w, pf.ps0, pf.ps1);
    }
    {   // blocks 4j+2, 4j+3
        const uint4 mt = lds128(meta_quad + 128);
        const uint32_t X0 = prmt(W1, W2, 0x6341u), X2 = W2 >> 8;
        a[0] = value_code<0, CB>(X0);
        a[1] = value_code<3, CB>(X0);
        a[2] = value_code<6, CB>(X0);
        a[3] = value_code<1, CB>(W2);
        mma16816_zero(t, a, pf.b0, pf.b1);
        mma16816(t, a, pf.c0, pf.c1);
        affine_accumulate(o2, t, mt.x, mt.y, pf.ps0, pf.ps1);
        a[0] = value_code<4, CB>(W2);
        a[1] = value_code<7, CB>(W2);
        a[2] = value_code<2, CB>(X2);
        a[3] = value_code<5, CB>(X2);
        mma16816_zero(t, a, pf.b0, pf.b1);
        mma16816(t, a, pf.c0, pf.c1);
        affine_accumulate(o3, t, mt.z, mt.w, pf.ps0, pf.ps1);
    }
}

// ---- record format 2 ---------------------------------------------------------------------------------
// The key levels of format 2 are eighths of small integers (2, 6, 11, 18), and four consecutive dims of a
// token are the four nibbles of one half-word: one byte-table lookup turns four codes into four signed bytes,
// and the products run as integer MMAs with the roles swapped: A = the rotated query (16 rows = 8 heads x 2
// of its 3 digits per MMA), B = the keys of eight tokens (32 dims per step).  S[head g][tokens 2tq, 2tq+1]
// then sits in the lane that needs exactly these probabilities as the B fragment of the value product: no
// transposition.
//
// Rotated query of head h: q' = delta_h (2^14 t0 + 2^7 t1 + t2), digits in [-64, 63], delta_h = max|q'| / (63 2^14):
// 21 bits below the largest coordinate (one fp16, 11 bits, is not enough for the 2e-3 bound; two int8 digits,
// 15 bits, fail it on short peaked rows by simulation).  The integer sums are exact.

// Two 32-dim steps (2j, 2j+1) of a Stale page: word triple (A, B, C) of the lane -> eight B registers
// (step, token half u, K half), then per step and token half one MMA for digits 0,1 and one for digit 2.
// q_pair: shared-memory address of this lane's query fragments of step 2j (digits 0,1 at +0, digit 2 at +512,
// step 2j+1 at +1024).
template <bool FIRST>      // FIRST: the page's first two steps start the four sums
__device__ __forceinline__ void tq3_key_pair_v2(int (&Sa0)[4], int (&Sb0)[4], int (&Sa1)[4], int (&Sb1)[4],
                                                uint32_t A, uint32_t Bw, uint32_t Cw, uint32_t q_pair)
{
    // signed levels +-{2, 6, 11, 18} (eight times the codebook) as bytes, indexed by code = magnitude | sign << 2
    constexpr uint32_t T0 = 0x120B0602u, T1 = 0xEEF5FAFEu;
    uint32_t sel[4], r[8];
    sel[0] = A & 0x77777777u;
    sel[1] = Bw & 0x77777777u;
    sel[2] = lop3_and_or(A >> 1, 0x44444444u, Cw & 0x33333333u);
    sel[3] = lop3_and_or(Bw >> 1, 0x44444444u, (Cw >> 2) & 0x33333333u);
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        r[2 * w] = prmt(T0, T1, sel[w]);
        r[2 * w + 1] = prmt(T0, T1, sel[w] >> 16);
    }
#pragma unroll
    for (int st = 0; st < 2; ++st) {
        // (the second fragment's rows 8-15 are stored as zeros: a full 16-byte load keeps the four operand
        // registers together, where building {x, 0, y, 0} cost two moves per MMA)
        const uint4 qa = lds128(q_pair + st * 1024), qb = lds128(q_pair + st * 1024 + 512);
        if (FIRST && st == 0) {
            mma16832_s8_zero(Sa0, qa.x, qa.y, qa.z, qa.w, r[0], r[1]);
            mma16832_s8_zero(Sb0, qb.x, qb.y, qb.z, qb.w, r[0], r[1]);
            mma16832_s8_zero(Sa1, qa.x, qa.y, qa.z, qa.w, r[2], r[3]);
            mma16832_s8_zero(Sb1, qb.x, qb.y, qb.z, qb.w, r[2], r[3]);
            continue;
        }
        mma16832_s8(Sa0, qa.x, qa.y, qa.z, qa.w, r[4 * st], r[4 * st + 1]);
        mma16832_s8(Sb0, qb.x, qb.y, qb.z, qb.w, r[4 * st], r[4 * st + 1]);
        mma16832_s8(Sa1, qa.x, qa.y, qa.z, qa.w, r[4 * st + 2], r[4 * st + 3]);
        mma16832_s8(Sb1, qb.x, qb.y, qb.z, qb.w, r[4 * st + 2], r[4 * st + 3]);
    }
}

// head g, one token: exact integer sums of the three digits -> the score in units of delta_h / 8
__device__ __forceinline__ float digits_to_score(int hi, int mid, int lo)
{
    return fmaf((float)hi, 16384.f, (float)(mid * 128 + lo));
}

// row form of the maximum from the column form and back (lanes 4h .. 4h+3 hold head h's row value; lane
// (g, tq) holds the column values of heads 2tq, 2tq+1)
template <int NB>
__device__ __forceinline__ void max_rows_from_columns(WarpAcc<NB>& acc, int lane)
{
    const int g = lane >> 2;
    const float a = __shfl_sync(0xffffffffu, acc.m[0], g >> 1), b = __shfl_sync(0xffffffffu, acc.m[1], g >> 1);
    acc.mr = (g & 1) ? b : a;
}

// Scores s[0..1] = tokens 2tq, 2tq+1, s[2..3] = tokens 2tq+8, 2tq+9, all of head g.  Raises the running
// maximum of head g when it is exceeded by more than the slack and rescales the accumulator columns.
template <int NB, bool TILED = false>
__device__ __forceinline__ void softmax_rescale_v2(WarpAcc<NB>& acc, const float (&s)[4], int lane)
{
    constexpr uint32_t FULL = 0xffffffffu;
    float mx = fmaxf(fmaxf(s[0], s[1]), fmaxf(s[2], s[3]));
    if (__any_sync(FULL, mx > acc.mr + kRescaleSlack)) {
        mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 2));
        const bool up = mx > acc.mr + kRescaleSlack;
        const float f = up ? fast_exp2(acc.mr - mx) : 1.f;
        if (up) acc.mr = mx;
        const int tq = lane & 3;
        const float f0 = __shfl_sync(FULL, f, 8 * tq), f1 = __shfl_sync(FULL, f, 8 * tq + 4);
        acc.m[0] = __shfl_sync(FULL, acc.mr, 8 * tq);
        acc.m[1] = __shfl_sync(FULL, acc.mr, 8 * tq + 4);
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            acc.o[i][0] *= f0; acc.o[i][2] *= f0;
            acc.o[i][1] *= f1; acc.o[i][3] *= f1;
        }
        acc.l[0] *= f0;
        acc.l[1] *= f1;
        if constexpr (TILED) {
            acc.lp[0] *= f0; acc.lp[1] *= f1;
            acc.pk[0] *= f0; acc.pk[1] *= f1;
        }
    }
}

// P of head g for the lane's four tokens is the B fragment of the value product as it stands.
template <int NB>
__device__ __forceinline__ void softmax_probs_v2(WarpAcc<NB>& acc, const float (&s)[4], PFrag& pf)
{
    const float p0 = fast_exp2(s[0] - acc.mr), p1 = fast_exp2(s[1] - acc.mr);
    const float p2 = fast_exp2(s[2] - acc.mr), p3 = fast_exp2(s[3] - acc.mr);
    pf.b0 = pack_f16x2(p0, p1);
    pf.b1 = pack_f16x2(p2, p3);
    const float2 h01 = half2_to_float2(pf.b0), h23 = half2_to_float2(pf.b1);
    pf.c0 = pack_f16x2(p0 - h01.x, p1 - h01.y);
    pf.c1 = pack_f16x2(p2 - h23.x, p3 - h23.y);
    const uint32_t ones[4] = {0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u};
    float ps[4];
    mma16816_zero(ps, ones, pf.b0, pf.b1);
    mma16816(ps, ones, pf.c0, pf.c1);
    pf.ps0 = ps[0];
    pf.ps1 = ps[1];
    acc.l[0] += ps[0];
    acc.l[1] += ps[1];
}

// Software-pipelined step over Stale pages: the value phase of the current page (record rec_v, its
// probabilities pf) and the score phase of the next page (record rec_k) are issued quad by quad in
// one instruction stream, so that table lookups, half-precision FMAs, fp32 FMAs and MMAs of the two
// phases overlap.  DO_V / DO_K switch the halves off for the first and the last page.
template <int D, bool DO_V, bool DO_K, bool DEFER = false, int FMT = 1>
__device__ __forceinline__ void tq3_step(WarpAcc<D / 16>& acc, uint32_t rec_v, const float (&s_cur)[4], PFrag& pf, uint32_t rec_k,
                                         uint32_t qt_lane, float sc2, int lane, float (&s_next)[4])
{
    constexpr int NB = D / 16, LW = 3 * NB / 4;
    const int g = lane >> 2;
    uint32_t kw[LW], vw[LW];
    float S0[4] = {0.f, 0.f, 0.f, 0.f}, S1[4] = {0.f, 0.f, 0.f, 0.f};
    int I0[4], I1[4], I2[4], I3[4];     // format 2: (digits 0,1 | 2) x (tokens g | g+8), started by the first pair of steps
    if constexpr (DO_K) load_lane_words<D>(rec_k, lane, kw);
    if constexpr (DO_V) load_lane_words<D>(rec_v + 6 * D, lane, vw);
    if constexpr (DO_V) {      // in one block with the key unpack of the next page
        if constexpr (FMT == 2) softmax_probs_v2<NB>(acc, s_cur, pf);
        else softmax_probs<NB>(acc, s_cur, pf);
    }
    if constexpr (DO_V && DEFER) {
        acc.lp[0] += pf.ps0;
        acc.lp[1] += pf.ps1;
    }
    const uint32_t meta = rec_v + 12 * D + 32 + g * 16;
#pragma unroll
    for (int j = 0; j < NB / 4; ++j) {
        if constexpr (DO_K) {
            if constexpr (FMT == 2) {
                if (j == 0) tq3_key_pair_v2<true>(I0, I1, I2, I3, kw[0], kw[1], kw[2], qt_lane);
                else tq3_key_pair_v2<false>(I0, I1, I2, I3, kw[3 * j], kw[3 * j + 1], kw[3 * j + 2], qt_lane + j * 2048);
            }
            else tq3_key_quad(S0, S1, kw[3 * j], kw[3 * j + 1], kw[3 * j + 2], qt_lane + j * 2048);
        }
        if constexpr (DO_V)
            tq3_value_quad<DEFER, FMT == 2>(acc.o[4 * j], acc.o[4 * j + 1], acc.o[4 * j + 2], acc.o[4 * j + 3], vw[3 * j], vw[3 * j + 1],
                                  vw[3 * j + 2], meta + j * 256, pf);
    }
    if constexpr (DO_K && FMT == 2) {
        // head g, tokens 2tq, 2tq+1 (I0 | I1) and 2tq+8, 2tq+9 (I2 | I3): the three query digits, then the token's
        // norm correction
        const int tq = lane & 3;
        const uint32_t gaddr = rec_k + 12 * D + 4 * tq;
        const float2 ga = half2_to_float2(lds32(gaddr)), gb = half2_to_float2(lds32(gaddr + 16));
        // (sc2 carries the head's digit unit delta_h / 8 here)
        s_next[0] = digits_to_score(I0[0], I0[2], I1[0]) * (ga.x * sc2);
        s_next[1] = digits_to_score(I0[1], I0[3], I1[1]) * (ga.y * sc2);
        s_next[2] = digits_to_score(I2[0], I2[2], I3[0]) * (gb.x * sc2);
        s_next[3] = digits_to_score(I2[1], I2[3], I3[1]) * (gb.y * sc2);
    }
    if constexpr (DO_K && FMT == 1) {
        const uint32_t gaddr = rec_k + 12 * D;
        const float r0 = __half2float(__ushort_as_half(lds16(gaddr + 2 * g))) * sc2;
        const float r1 = __half2float(__ushort_as_half(lds16(gaddr + 2 * g + 16))) * sc2;
        s_next[0] = (S0[0] + S1[0]) * r0;
        s_next[1] = (S0[1] + S1[1]) * r0;
        s_next[2] = (S0[2] + S1[2]) * r1;
        s_next[3] = (S0[3] + S1[3]) * r1;
    }
}

// Four 8x8 matrices of 16-bit elements from shared memory in the MMA fragment layout: lane l supplies the
// address of row l % 8 of matrix l / 8; every lane receives, per matrix, the 32 bits at (row lane / 4,
// 16-bit columns 2 (lane % 4), 2 (lane % 4) + 1).
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

// One Recent/Anchor page: keys [16 tokens][d] e4m3 at kaddr, values [d channels][16 tokens] at vaddr.
// MMA row r of the score tile holds token pi(r) = 4 (r % 8 / 2) + r % 2 + 2 (r / 8), so that the value
// fragments can be fetched with ldmatrix: a lane then holds the four consecutive tokens 4tq .. 4tq+3 of
// its two channel rows, which is the order P^T has after the transposition of a score tile whose rows
// are permuted this way.
template <int D, bool SCORED, bool ACCUMULATE = false>
__device__ __forceinline__ void fp8_page(WarpAcc<D / 16>& acc, uint32_t kaddr, uint32_t vaddr, uint32_t qf_lane,
                                         float score_scale, float v_scale, int valid, int lane, float* mass_pg,
                                         int mass_stride, int GQ)
{
    constexpr int NB = D / 16;
    const int g = lane >> 2, tq = lane & 3;
    const int tok0 = 4 * (g >> 1) + (g & 1), tok1 = tok0 + 2;       // tokens of the lane's two score rows
    float S0[4] = {0.f, 0.f, 0.f, 0.f}, S1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < D / 64; ++j) {
        const uint4 r0 = lds128(kaddr + tok0 * D + 64 * j + 16 * tq);
        const uint4 r1 = lds128(kaddr + tok1 * D + 64 * j + 16 * tq);
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
    float s[4] = {(S0[0] + S1[0]) * score_scale, (S0[1] + S1[1]) * score_scale, (S0[2] + S1[2]) * score_scale,
                  (S0[3] + S1[3]) * score_scale};
    // bytes of tokens beyond the sequence end are cleared so that stale NaN patterns cannot leak
    uint32_t keep = 0xFFFFFFFFu;                     // byte mask for the tokens 4tq .. 4tq+3 of a value word
    if (valid < kPage) {
        if (tok0 >= valid) s[0] = s[1] = -CUDART_INF_F;
        if (tok1 >= valid) s[2] = s[3] = -CUDART_INF_F;
        keep = (4 * tq < valid ? 0x000000FFu : 0u) | (4 * tq + 1 < valid ? 0x0000FF00u : 0u) |
               (4 * tq + 2 < valid ? 0x00FF0000u : 0u) | (4 * tq + 3 < valid ? 0xFF000000u : 0u);
    }
    PFrag pf;
    softmax_page<NB>(acc, s, pf);
    if constexpr (SCORED) store_page_mass<NB, ACCUMULATE>(acc, pf.ps0, pf.ps1, mass_pg, mass_stride, GQ, lane);
    const bool scale_v = v_scale != 1.0f;
#pragma unroll
    for (int cb = 0; cb < NB; cb += 2) {
        // channels 16cb .. 16cb+31: rows of 16 bytes, lane l addresses row l
        uint32_t v[4];
        ldmatrix_x4(vaddr + cb * 256 + lane * 16, v[0], v[1], v[2], v[3]);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const uint32_t lo = v[2 * e] & keep, hi = v[2 * e + 1] & keep;      // channel rows g and g + 8 of block cb + e
            uint32_t a[4];
            a[0] = e4m3x2_to_f16x2((uint16_t)(lo & 0xFFFFu));
            a[1] = e4m3x2_to_f16x2((uint16_t)(hi & 0xFFFFu));
            a[2] = e4m3x2_to_f16x2((uint16_t)(lo >> 16));
            a[3] = e4m3x2_to_f16x2((uint16_t)(hi >> 16));
            if (scale_v) {
                float t[4];
                mma16816_zero(t, a, pf.b0, pf.b1);
                mma16816(t, a, pf.c0, pf.c1);
#pragma unroll
                for (int i = 0; i < 4; ++i) acc.o[cb + e][i] = fmaf(v_scale, t[i], acc.o[cb + e][i]);
            } else {
                mma16816(acc.o[cb + e], a, pf.b0, pf.b1);
                mma16816(acc.o[cb + e], a, pf.c0, pf.c1);
            }
        }
    }
}

// Eq. (softmax-merge) of one (request, KV head) row that was split over n_parts blocks.  Part 0 sits
// in slot first_slot, part j > 0 in slot even_base + 2j.  Called by all NT threads of the block that
// drew the row's last ticket; `buf` is idle shared memory (n_parts * 16 + 16 floats).  Warp hd < 8
// reduces the maxima and row sums of head hd (one trip to L2: both are loaded together and kept in
// shared memory); a thread then owns float4 groups (one channel, four heads) of the [channel][8 heads]
// tile and has 40 loads in flight, issued before the weights are worked out.
template <int D, int NT, int KPMAX = 40>
__device__ __forceinline__ void merge_row(const DecodeParams& P, int first_slot, int even_base, int n_parts,
                                          float* buf, int b, int h)
{
    constexpr uint32_t FULL = 0xffffffffu;
    constexpr int STRIDE = 8 * D + 16, GPT = (2 * D + NT - 1) / NT, KP = KPMAX / GPT;   // KPMAX (40) float4 loads in flight per thread
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int GQ = P.group, hq = P.hkv * GQ;
    float* w_s = buf;                        // [n_parts][8] maxima, then weights e^{m_j - m}
    float* l_s = buf + n_parts * 8;          // [n_parts][8] row sums
    float* ml_s = buf + n_parts * 16;        // [8] m, [8] l of the row
    auto slot_of = [&](int j) -> const float* {
        return P.partials + (size_t)(j == 0 ? first_slot : even_base + 2 * j) * STRIDE;
    };
    __syncthreads();
    float4 acc[GPT], v[KP][GPT];
#pragma unroll
    for (int k = 0; k < GPT; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    const int head0 = (tid & 1) * 4;         // NT is even: every group of this thread covers the same four heads
    auto load_round = [&](int j0) {
#pragma unroll
        for (int p = 0; p < KP; ++p) {
            const float* ps = slot_of(min(j0 + p, n_parts - 1));
#pragma unroll
            for (int k = 0; k < GPT; ++k)
                v[p][k] = __ldcg(reinterpret_cast<const float4*>(ps) + min(tid + k * NT, 2 * D - 1));
        }
    };
    auto use_round = [&](int j0) {
#pragma unroll
        for (int p = 0; p < KP; ++p)
            if (j0 + p < n_parts) {
                const float4 w = *reinterpret_cast<const float4*>(w_s + (j0 + p) * 8 + head0);
#pragma unroll
                for (int k = 0; k < GPT; ++k) {
                    acc[k].x = fmaf(w.x, v[p][k].x, acc[k].x);
                    acc[k].y = fmaf(w.y, v[p][k].y, acc[k].y);
                    acc[k].z = fmaf(w.z, v[p][k].z, acc[k].z);
                    acc[k].w = fmaf(w.w, v[p][k].w, acc[k].w);
                }
            }
    };
    load_round(0);                           // in flight while the weights are worked out
    for (int hd = warp; hd < 8; hd += NT / 32) {
        float M = -CUDART_INF_F;
        for (int j = lane; j < n_parts; j += 32) {
            const float* ps = slot_of(j) + 8 * D;
            const float lj = __ldcg(ps + 8 + hd), mj = __ldcg(ps + hd);
            l_s[j * 8 + hd] = lj;
            w_s[j * 8 + hd] = mj;
            if (lj > 0.f) M = fmaxf(M, mj);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(FULL, M, o));
        float L = 0.f;
        for (int j = lane; j < n_parts; j += 32) {      // re-reads this lane's own entries
            const float lj = l_s[j * 8 + hd];
            const float w = lj > 0.f ? fast_exp2(w_s[j * 8 + hd] - M) : 0.f;
            w_s[j * 8 + hd] = w;
            L = fmaf(w, lj, L);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(FULL, L, o);
        if (lane == 0) {
            ml_s[hd] = M;
            ml_s[8 + hd] = L;
        }
    }
    __syncthreads();
    use_round(0);
    for (int j0 = KP; j0 < n_parts; j0 += KP) {
        load_round(j0);
        use_round(j0);
    }
#pragma unroll
    for (int k = 0; k < GPT; ++k) {
        const int grp = tid + k * NT, ch = grp >> 1;
        if (grp >= 2 * D) continue;
        const float av[4] = {acc[k].x, acc[k].y, acc[k].z, acc[k].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int head = head0 + e;
            if (head < GQ) {
                const float L = ml_s[8 + head];
                P.out[((size_t)b * hq + h * GQ + head) * D + ch] = L > 0.f ? av[e] / L : 0.f;
            }
        }
    }
    if (P.lse && tid < GQ)
        P.lse[(size_t)b * hq + h * GQ + tid] = ml_s[8 + tid] > 0.f ? (ml_s[tid] + log2f(ml_s[8 + tid])) * kLn2 : -CUDART_INF_F;
}

template <int D, int NW, int NSTAGE, int MINB, bool SCORED, bool TILED, int MAXL, int FMT>
__global__ void __launch_bounds__(NW * 32, MINB) decode_tensor_kernel(const LayerSet<MAXL> LS)
{
    const DecodeParams& P0 = LS.layer[0];    // requests and geometry are common to all layers
    using G = Geo<D, NW, NSTAGE, TILED>;     // pages of several tiles: short rounds leave room for the parked rows
    constexpr int NB = G::NB, NBH = NB, NU = NW;
    constexpr uint32_t FULL = 0xffffffffu;
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    int* cum = reinterpret_cast<int*>(smem + G::OFF_CUM);
    int* strides = reinterpret_cast<int*>(smem + G::OFF_STRIDE);
    float* sm_m = reinterpret_cast<float*>(smem + G::OFF_M);
    float* sm_l = reinterpret_cast<float*>(smem + G::OFF_L);
    Partition* pt = reinterpret_cast<Partition*>(smem + G::OFF_PART);
    int* last_s = reinterpret_cast<int*>(smem + G::OFF_LAST);
    float* red = reinterpret_cast<float*>(smem);            // [NW][D][8] over the ring, between segments

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    const int unit = warp, hf = 0;
    const int hkv = P0.hkv, GQ = P0.group, hq = hkv * GQ;
    const int n_layers = MAXL == 1 ? 1 : LS.n;
    // a length beyond the table row is cut to the row (and flagged), so that no entry past it is ever read
    const int len_cap = P0.max_pages * P0.tiles * kPage;
    auto length_of = [&](int b) -> int {
        const int len = P0.lens[b];
        if (len > len_cap) {
            atomicOr(P0.status, kStBounds);
            return len_cap;
        }
        return len < 0 ? 0 : len;
    };

    // ---- prologue: barriers, prefix of pages, page strides ---------------------------------------
    if (tid == 0) {
        for (int i = 0; i < NW * NSTAGE; ++i) mbar_init(sbase + G::OFF_BAR + 8 * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        last_s[1] = 0;
    }
    if (warp == 0) {
        int run = 0;
        for (int b0 = 0; b0 < P0.B; b0 += 32) {
            const int b = b0 + lane;
            int n = 0;
            if (b < P0.B) {
                const int len = length_of(b);
                n = len > 0 ? ((len + kPage - 1) / kPage) * hkv : 0;
            }
            int inc = n;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(FULL, inc, o);
                if (lane >= o) inc += v;
            }
            if (b < P0.B) cum[b] = run + inc - n;
            run += __shfl_sync(FULL, inc, 31);
        }
        if (lane == 0) cum[P0.B] = run;
        __syncwarp();
        build_partition(pt, cum, P0.B, hkv, gridDim.x, lane);
    } else {
        // Pages of a row are visited in a strided order, page(i) = i * stride mod n_pages, the stride
        // coprime to n_pages and near 0.618 n_pages: every contiguous range of positions then holds the
        // row's FP8 and TQ3 pages in their overall proportion, so equal ranges cost equal time.
        for (int b = tid - 32; b < P0.B; b += NW * 32 - 32) {
            const int len = length_of(b), n = (len + kPage - 1) / kPage;
            int st = (int)((float)n * 0.6180339f);
            if (st < 1) st = 1;
            if constexpr (TILED) st = 1;          // consecutive tiles: a warp's run stays inside one or two pages
            for (; n > 1 && !TILED; ++st) {
                int a = st, c = n;
                while (c) { const int t = a % c; a = c; c = t; }
                if (a == 1) break;
            }
            strides[b] = st;
        }
    }
    __syncthreads();
    int my_start = 0, my_end = 0;                          // more blocks than work: an empty range
    if ((int)blockIdx.x < pt->blocks) partition_range(pt, cum, hkv, P0.B, blockIdx.x, my_start, my_end);

    // per-warp ring of NSTAGE slots; one bit per slot holds the mbarrier phase the next wait must see
    uint32_t phase = 0;
    bool failed = false;
    const uint32_t ring = sbase + warp * NSTAGE * G::SLOT;
    const uint32_t bars = sbase + G::OFF_BAR + warp * NSTAGE * 8;
    const uint32_t qt_lane = sbase + G::OFF_QT + lane * 16, qf_lane = sbase + G::OFF_QF + lane * 8;
    int* list3 = reinterpret_cast<int*>(smem + G::OFF_LIST) + warp * 2 * G::ROUND;   // Stale page ids of the round
    int* list8 = list3 + G::ROUND;                                                   // FP8 page ids | valid << 27
    int* lpg3 = reinterpret_cast<int*>(smem + G::OFF_LIST) + (NW + warp) * 2 * G::ROUND;   // their logical pages (scored variant)
    int* lpg8 = lpg3 + G::ROUND;
    const float sc2 = P0.scale * kLog2e;     // scores are kept in log2 units
    uint32_t pending = 0;                    // ring slots with a copy in flight that nobody has waited for yet
    // Bounded wait for ring slot s, then flip its expected phase.  `limit_ns` of wall time (the pool's wait
    // limit, 20 ms by default); returns false when it ran out.
    auto wait_bounded = [&](uint32_t s, unsigned long long limit_ns) -> bool {
        const uint32_t bar = bars + 8 * s, parity = (phase >> s) & 1u;
        // limit 0 (diagnostic): one look without blocking, so that a copy still in flight counts as late
        bool ok = limit_ns == 0 ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity);
        if (!ok && limit_ns != 0) {
            unsigned long long t0, t1;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
            for (int spins = 1; !ok; ++spins) {
                ok = mbar_try_wait(bar, parity);
                if (!ok && (spins & 255) == 0) {
                    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
                    if (t1 - t0 >= limit_ns) break;
                }
            }
        }
        ok = __all_sync(FULL, ok);           // the copy has landed for every lane, or the warp gives up as one
        if (ok) {
            phase ^= 1u << s;
            pending &= ~(1u << s);
        }
        return ok;
    };
    // After a wait has run out the warp stops scanning; before anybody reuses the ring (as the reduction
    // buffer) or the block leaves, every copy this warp still has in flight is waited for with the
    // default limit, so that nothing lands in memory that has changed hands.
    auto drain = [&]() {
        bool lost = false;
#pragma unroll 1
        for (uint32_t s = 0; s < (uint32_t)NSTAGE; ++s)
            if (pending & (1u << s)) lost |= !wait_bounded(s, kDefaultWaitNs);
        return lost;
    };

    for (int layer = 0; layer < n_layers; ++layer) {
    const DecodeParams& P = LS.layer[MAXL == 1 ? 0 : layer];
    auto wait_slot = [&](uint32_t s) {
        if (!wait_bounded(s, P.wait_ns)) {
            failed = true;
            atomicOr(P.status, kStTimeout);
        }
    };
    // rows of empty requests
    for (int b = blockIdx.x; b < P.B; b += gridDim.x)
        if (P.lens[b] <= 0) {
            for (int i = tid; i < hq * D; i += NW * 32) P.out[(size_t)b * hq * D + i] = 0.f;
            if (P.lse)
                for (int i = tid; i < hq; i += NW * 32) P.lse[(size_t)b * hq + i] = -CUDART_INF_F;
        }

    int pos = my_start;
    int b = 0;
    while (pos < my_end) {
        // ---- locate the segment: request b, KV head h, positions [pg0, pg0 + n_seg) of the row ------
        while (cum[b + 1] <= pos) ++b;
        const int len = min(max(P.lens[b], 0), len_cap), n_pages = (len + kPage - 1) / kPage;
        const int h = (pos - cum[b]) / n_pages, pg0 = (pos - cum[b]) % n_pages;
        const int row_start = cum[b] + h * n_pages, row_end = row_start + n_pages;
        const int n_seg = min(my_end, row_end) - pos;
        const int32_t* bt_row = P.bt + (size_t)b * P.max_pages;
        const uint8_t* tag_row = P.tags + (size_t)b * P.max_pages;
        // this warp's pages: a contiguous run of positions (a run of the strided order holds FP8 and TQ3
        // pages in the row's proportion, so the warps of a block finish together)
        const int warp_first = (int)(((unsigned)n_seg * (unsigned)warp) / NW);
        const int n_my = (int)(((unsigned)n_seg * (unsigned)(warp + 1)) / NW) - warp_first;
        const int stride = strides[b];
        constexpr int EPL = D / 32;
        constexpr int HPW = (8 + NW - 1) / NW;      // query heads a warp prepares (head warp, warp + NW, ...)
        float qx[HPW][EPL];       // loaded before anything else waits
#pragma unroll
        for (int k = 0; k < HPW; ++k)
#pragma unroll
            for (int r = 0; r < EPL; ++r) {
                const int hd = warp + k * NW;
                qx[k][r] = (hd < GQ) ? __bfloat162float(P.q[((size_t)b * hq + h * GQ + hd) * D + lane * EPL + r]) : 0.f;
            }
        float* mass_row = SCORED ? P.mass + ((size_t)b * hq + (size_t)h * GQ) * P.max_pages : nullptr;
        const uint8_t* tq3_base = P.tq3 + (size_t)h * G::TQ3_REC;
        const uint8_t* fp8_base = P.fp8 + (size_t)h * (2 * G::FP8_HALF);
        // pages of several tiles: a TQ3 page is tiles * (12 D + 32) bytes of tiles, then 4 D bytes of value
        // scale/zero shared by its tiles; an FP8 page is `tiles` consecutive 16-token records
        constexpr int TQ3_TILE = 12 * D + 32, TQ3_META = 4 * D;
        const size_t tq3_page = (size_t)P.tiles * TQ3_TILE + TQ3_META;

        // Table entries of up to G::ROUND of the warp's pages are compacted into two id lists, one per
        // format (entry i of a 32-page chunk is read by lane i; ballots give the positions).
        int n3 = 0, n8 = 0;
        auto build_lists = [&](int round) {
            n3 = n8 = 0;
#pragma unroll 1
            for (int c = 0; c < G::ROUND / 32; ++c) {
                const int i = round * G::ROUND + c * 32 + lane;
                int kind = 0, id = 0, valid = kPage, pg = 0;
                if (i < n_my) {
                    pg = (int)(((unsigned)(pg0 + warp_first + i) * (unsigned)stride) % (unsigned)n_pages);   // < 2^32: max_pages <= 65535
                    // `pg` counts 16-token tiles of the row; the table has one entry per page of P.tiles tiles
                    const int entry = TILED ? pg / P.tiles : pg;
                    id = bt_row[entry];
                    const int tag = tag_row[entry];
                    valid = min(kPage, len - pg * kPage);
                    if (tag == MKV_TAG_STALE)
                        kind = (id >= 0 && id < P.tq3_pages && valid == kPage) ? 1 : 0;
                    else
                        kind = (tag <= MKV_TAG_ANCHOR && id >= 0 && id < P.fp8_pages) ? 2 : 0;
                    if (kind == 0) atomicOr(P.status, kStBounds);     // never dereferenced
                    if constexpr (TILED) pg = (pg - entry * P.tiles) | (entry << 16);   // second list: tile inside its page | logical page << 16
                }
                const uint32_t m3 = __ballot_sync(FULL, kind == 1), m8 = __ballot_sync(FULL, kind == 2);
                const uint32_t lt = (1u << lane) - 1u;
                if (kind == 1) list3[n3 + __popc(m3 & lt)] = id;
                if (kind == 2) list8[n8 + __popc(m8 & lt)] = id | ((valid & 15) << 27);
                if constexpr (SCORED || TILED) {     // logical page (scored output) or tile inside the page (pages of several tiles)
                    if (kind == 1) lpg3[n3 + __popc(m3 & lt)] = pg;
                    if (kind == 2) lpg8[n8 + __popc(m8 & lt)] = pg;
                }
                n3 += __popc(m3);
                n8 += __popc(m8);
            }
            __syncwarp();
        };
        auto issue_tq3 = [&](int i) {      // copy Stale page i of the round into ring slot i % NSTAGE
            pending |= 1u << ((uint32_t)i % NSTAGE);
            if (lane == 0) {
                const uint32_t s = (uint32_t)i % NSTAGE;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                if constexpr (!TILED) {
                    mbar_expect_tx(bars + 8 * s, G::TQ3_REC);
                    bulk_load(ring + s * G::SLOT, tq3_base + (size_t)list3[i] * hkv * G::TQ3_REC, G::TQ3_REC, bars + 8 * s);
                } else {   // the tile only: the page's scale/zero are applied once, when the scan leaves the page
                    const int page = list3[i], m = lpg3[i] & 0xFFFF;
                    const uint8_t* pbase = P.tq3 + ((size_t)page * hkv + h) * tq3_page;
                    mbar_expect_tx(bars + 8 * s, TQ3_TILE);
                    bulk_load(ring + s * G::SLOT, pbase + (size_t)m * TQ3_TILE, TQ3_TILE, bars + 8 * s);
                }
            }
        };
        auto issue_fp8 = [&](int i) {      // copy FP8 page i of the round into the slot pair 2 (i % (NSTAGE/2))
            pending |= 3u << ((uint32_t)(2 * i) % NSTAGE);
            if (lane == 0) {
                const uint32_t s = (uint32_t)(2 * i) % NSTAGE;
                const int e8 = list8[i] & 0x7FFFFFF;
                const uint8_t* rec;
                if constexpr (!TILED) {
                    rec = fp8_base + (size_t)e8 * hkv * (2 * G::FP8_HALF);
                } else {
                    rec = P.fp8 + (((size_t)e8 * hkv + h) * P.tiles + (lpg8[i] & 0xFFFF)) * (2 * G::FP8_HALF);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_expect_tx(bars + 8 * s, G::FP8_HALF);
                bulk_load(ring + s * G::SLOT, rec, G::FP8_HALF, bars + 8 * s);
                mbar_expect_tx(bars + 8 * (s + 1), G::FP8_HALF);
                bulk_load(ring + (s + 1) * G::SLOT, rec + G::FP8_HALF, G::FP8_HALF, bars + 8 * (s + 1));
            }
        };

        WarpAcc<NB> acc;
        // Pages of several tiles.  While the scan is inside a Stale page, acc.o holds sum p * code and the
        // output gathered before waits in this warp's shared-memory rows ("parked"); leaving the page adds
        // scale * acc.o + zero * acc.lp to it (fold).  The scale/zero halves come straight from the page's
        // metadata in global memory, in the order of the 16-token record.
        float* park = reinterpret_cast<float*>(smem + G::SMEM) + (size_t)warp * NB * 128;
        auto park_store = [&]() {
#pragma unroll
            for (int i = 0; i < NB; ++i)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    park[(i * 4 + e) * 32 + lane] = acc.o[i][e];
                    acc.o[i][e] = 0.f;
                }
            acc.pk[0] = acc.pk[1] = 1.f;
            acc.lp[0] = acc.lp[1] = 0.f;
        };
        auto fold = [&](int page, bool to_regs, int logical_page) {
            if constexpr (SCORED)      // this warp's part of the page's exponential sum
                store_page_mass<NB, true>(acc, acc.lp[0], acc.lp[1], mass_row + logical_page, P.max_pages, GQ, lane);
            const uint4* meta = reinterpret_cast<const uint4*>(P.tq3 + ((size_t)page * hkv + h) * tq3_page +
                                                                (size_t)P.tiles * TQ3_TILE + g * 16);
#pragma unroll
            for (int j = 0; j < NB / 4; ++j) {
                const uint4 m01 = __ldg(meta + j * 16), m23 = __ldg(meta + j * 16 + 8);
                const uint32_t scp[4] = {m01.x, m01.z, m23.x, m23.z}, zpp[4] = {m01.y, m01.w, m23.y, m23.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int i = 4 * j + q;
                    const float2 sc = half2_to_float2(scp[q]), zp = half2_to_float2(zpp[q]);
                    float r[4];
                    r[0] = fmaf(park[(i * 4 + 0) * 32 + lane], acc.pk[0], fmaf(sc.x, acc.o[i][0], zp.x * acc.lp[0]));
                    r[1] = fmaf(park[(i * 4 + 1) * 32 + lane], acc.pk[1], fmaf(sc.x, acc.o[i][1], zp.x * acc.lp[1]));
                    r[2] = fmaf(park[(i * 4 + 2) * 32 + lane], acc.pk[0], fmaf(sc.y, acc.o[i][2], zp.y * acc.lp[0]));
                    r[3] = fmaf(park[(i * 4 + 3) * 32 + lane], acc.pk[1], fmaf(sc.y, acc.o[i][3], zp.y * acc.lp[1]));
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (to_regs) acc.o[i][e] = r[e];
                        else { park[(i * 4 + e) * 32 + lane] = r[e]; acc.o[i][e] = 0.f; }
                    }
                }
            }
            acc.pk[0] = acc.pk[1] = 1.f;
            acc.lp[0] = acc.lp[1] = 0.f;
        };
        (void)park_store; (void)fold;
#pragma unroll
        for (int i = 0; i < NB; ++i) acc.o[i][0] = acc.o[i][1] = acc.o[i][2] = acc.o[i][3] = 0.f;
        acc.l[0] = acc.l[1] = 0.f;
        acc.m[0] = acc.m[1] = -CUDART_INF_F;
        acc.mr = -CUDART_INF_F;

        // first round: start the copies, then build the query fragments while they fly
        const int n_rounds = (n_my + G::ROUND - 1) / G::ROUND;
        if (n_rounds > 0) {
            build_lists(0);
            for (int i = 0; i < min(n3, NSTAGE); ++i) issue_tq3(i);
        }

        // query fragments: a warp rotates head `warp` (and `warp + NW`); loads were issued before the copies started
#pragma unroll
        for (int k = 0; k < HPW; ++k) {
            const int hd = warp + k * NW;
            if (hd >= 8) break;
            float a[EPL];
#pragma unroll
            for (int r = 0; r < EPL; ++r) {
                const int i = lane * EPL + r;
                a[r] = ((P.sigma.w[i >> 5] >> (i & 31)) & 1u) ? -qx[k][r] : qx[k][r];
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
            __half* qf = reinterpret_cast<__half*>(smem + G::OFF_QF);
            if constexpr (FMT == 2) {
                // rotated query as three balanced base-128 digits in the A-fragment order of the integer key
                // products: dim i sits in step i/32 at K slot k = i%32 of fragment lane 4 hd + (k%16)/4, byte k%4;
                // digits 0,1 in registers 2 (k/16) + digit of the step's first 512 bytes, digit 2 in register 2 (k/16)
                // of the second 512 bytes, whose odd registers (fragment rows 8-15) are zero
                uint8_t* qt8 = smem + G::OFF_QT;
                float amax = 0.f;
#pragma unroll
                for (int r = 0; r < EPL; ++r) amax = fmaxf(amax, fabsf(a[r] * rs));
#pragma unroll
                for (int m = 16; m > 0; m >>= 1) amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, m));
                const float delta = amax > 0.f ? amax * (1.f / (63.f * 16384.f)) : 1.f, inv_delta = 1.f / delta;
                if (lane == 0) reinterpret_cast<float*>(smem + G::OFF_QS)[hd] = delta * 0.125f;   // key levels are eighths
#pragma unroll
                for (int r0 = 0; r0 < EPL; r0 += 4) {
                    uint32_t word[3] = {0u, 0u, 0u};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int Q = __float2int_rn(a[r0 + e] * rs * inv_delta);
                        const int t2 = ((Q + 64) & 127) - 64, Q1 = (Q - t2) >> 7;
                        const int t1 = ((Q1 + 64) & 127) - 64, t0 = (Q1 - t1) >> 7;
                        word[0] |= (uint32_t)(t0 & 0xFF) << (8 * e);
                        word[1] |= (uint32_t)(t1 & 0xFF) << (8 * e);
                        word[2] |= (uint32_t)(t2 & 0xFF) << (8 * e);
                    }
                    const int i0 = lane * EPL + r0, st = i0 >> 5, k = i0 & 31;
                    const int L = 4 * hd + ((k & 15) >> 2);
                    *reinterpret_cast<uint32_t*>(qt8 + ((st * 2) * 32 + L) * 16 + (2 * (k >> 4)) * 4) = word[0];
                    *reinterpret_cast<uint32_t*>(qt8 + ((st * 2) * 32 + L) * 16 + (2 * (k >> 4) + 1) * 4) = word[1];
                    *reinterpret_cast<uint2*>(qt8 + ((st * 2 + 1) * 32 + L) * 16 + (k >> 4) * 8) = make_uint2(word[2], 0u);
                }
            }
#pragma unroll
            for (int r = 0; r < EPL; ++r) {
                const int i = lane * EPL + r;
                if constexpr (FMT == 1) {   // rotated query, natural slot order: block i/16, slot s = i%16; per lane {hi b0, hi b1, lo b0, lo b1}
                    const int kb = i >> 4, s = i & 15;
                    const int at = (kb * 32 + 4 * hd + ((s & 7) >> 1)) * 8 + (s >> 3) * 2 + (s & 1);
                    // fp16 pair hi + lo carries the rotated query to ~2^-22
                    const float v = a[r] * rs;
                    const __half vh = __float2half_rn(v);
                    qt[at] = vh;
                    qt[at + 4] = __float2half_rn(v - __half2float(vh));
                }
                {   // plain query in the slot order of the FP8 key loads: 16 consecutive dims per lane
                    const int j = i >> 6, t4 = (i & 63) >> 4, wv = (i & 15) >> 2, e = i & 3;
                    qf[((4 * j + wv) * 32 + 4 * hd + t4) * 4 + (e >> 1) * 2 + (e & 1)] = __float2half_rn(qx[k][r]);
                }
            }
        }
        __syncthreads();
        // score unit of the Stale pages: record format 2 counts in digit units of this lane's head g
        const float sc2k = FMT == 2 ? sc2 * reinterpret_cast<const float*>(smem + G::OFF_QS)[g] : sc2;

        for (int round = 0; round < n_rounds && !failed; ++round) {
            if (round > 0) {
                build_lists(round);
                for (int i = 0; i < min(n3, NSTAGE); ++i) issue_tq3(i);
            }
            // ---- Stale pages: scores of page i+1 are computed together with the output update of page i
            if (n3 > 0) {
                float s_cur[4], s_next[4];
                PFrag pf;
                int cur_page = 0, cur_lp = 0;             // physical id and logical index of the Stale page being scanned
                if constexpr (TILED) {
                    park_store();
                    cur_page = list3[0];
                    cur_lp = lpg3[0] >> 16;
                }
                wait_slot(0);
                if (!failed) tq3_step<D, false, true, TILED, FMT>(acc, 0, s_cur, pf, ring, qt_lane, sc2k, lane, s_cur);
                for (int i = 0; i + 1 < n3 && !failed; ++i) {
                    const uint32_t cur = (uint32_t)i % NSTAGE, nxt = (uint32_t)(i + 1) % NSTAGE;
                    wait_slot(nxt);
                    if (failed) break;
                    if constexpr (FMT == 2) softmax_rescale_v2<NB, TILED>(acc, s_cur, lane);
                    else softmax_rescale<NB, TILED>(acc, s_cur);
                    if constexpr (TILED) {
                        const int pg_i = list3[i];
                        if (pg_i != cur_page) {
                            fold(cur_page, false, cur_lp);
                            cur_page = pg_i;
                            cur_lp = lpg3[i] >> 16;
                        }
                    }
                    tq3_step<D, true, true, TILED, FMT>(acc, ring + cur * G::SLOT, s_cur, pf, ring + nxt * G::SLOT, qt_lane, sc2k, lane, s_next);
                    if constexpr (SCORED && !TILED) store_page_mass<NB>(acc, pf.ps0, pf.ps1, mass_row + lpg3[i], P.max_pages, GQ, lane);
#pragma unroll
                    for (int e = 0; e < 4; ++e) s_cur[e] = s_next[e];
                    __syncwarp();
                    if (i + NSTAGE < n3) issue_tq3(i + NSTAGE);
                }
                if (!failed) {
                    if constexpr (FMT == 2) softmax_rescale_v2<NB, TILED>(acc, s_cur, lane);
                    else softmax_rescale<NB, TILED>(acc, s_cur);
                    if constexpr (TILED) {
                        const int pg_i = list3[n3 - 1];
                        if (pg_i != cur_page) {
                            fold(cur_page, false, cur_lp);
                            cur_page = pg_i;
                            cur_lp = lpg3[n3 - 1] >> 16;
                        }
                    }
                    tq3_step<D, true, false, TILED, FMT>(acc, ring + ((uint32_t)(n3 - 1) % NSTAGE) * G::SLOT, s_cur, pf, 0, qt_lane, sc2k, lane, s_next);
                    if constexpr (SCORED && !TILED) store_page_mass<NB>(acc, pf.ps0, pf.ps1, mass_row + lpg3[n3 - 1], P.max_pages, GQ, lane);
                    if constexpr (TILED) fold(cur_page, true, cur_lp);   // back to output units for the FP8 pages and the reduction
                }
                __syncwarp();
            }
            // ---- Recent/Anchor pages: two slots per page (keys, values)
            if (n8 > 0 && !failed) {
                for (int i = 0; i < min(n8, NSTAGE / 2); ++i) issue_fp8(i);
                for (int i = 0; i < n8 && !failed; ++i) {
                    const uint32_t s = (uint32_t)(2 * i) % NSTAGE;
                    wait_slot(s);
                    wait_slot(s + 1);
                    if (failed) break;
                    const int e = list8[i];
                    const int valid = (e >> 27) & 15;
                    fp8_page<D, SCORED, TILED>(acc, ring + s * G::SLOT, ring + (s + 1) * G::SLOT, qf_lane, sc2 * P.k_scale, P.v_scale,
                                               valid ? valid : kPage, lane,
                                               SCORED ? mass_row + (TILED ? (lpg8[i] >> 16) : lpg8[i]) : nullptr, P.max_pages, GQ);
                    if constexpr (FMT == 2) max_rows_from_columns<NB>(acc, lane);     // the page may have raised the maxima
                    __syncwarp();
                    if (i + NSTAGE / 2 < n8) issue_fp8(i + NSTAGE / 2);
                }
            }
        }
        float (&oacc)[NBH][4] = acc.o;
        float (&lacc)[2] = acc.l;
        float (&m_run)[2] = acc.m;

        // ---- combine the warps of the block (ring memory is idle now) ---------------------------
        if (failed && drain()) last_s[1] = 1;      // a copy never arrived at all: the block must not touch the ring
        __syncthreads();
        if (last_s[1]) return;                     // (the call has failed; its workspace needs mkv_workspace_init again)
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

        const bool whole_row = (pos == row_start) && (pos + n_seg == row_end);
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
            // partial (m, l, O) of this block for the row; slot 2c if the segment opens the block's range,
            // 2c + 1 otherwise
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
            // Ticket of the row (store -> fence -> ticket on the writers' side, ticket -> fence -> load on the
            // merger's).  Who merges?  In the last layer of the launch the block that draws the row's last
            // ticket.  In an earlier layer the row is left to the block that is FIRST to finish the same row in
            // the next layer -- the one that is ahead of the others, so that the merges do not keep falling on
            // the block that is already late.  That block finds the row complete and merges it, or it leaves a
            // request (the counter's top bit) and the row's last arrival, seeing the request, merges after all.
            // Either way exactly one block merges, and it leaves the counter at zero for the next call.
            int c0, c1;
            partition_blocks_of_row(pt, cum, P.B, b * hkv + h, row_start, row_end, c0, c1);
            const int n_parts = c1 - c0 + 1;
            constexpr uint32_t kRequest = 0x80000000u;
            __syncthreads();
            if (tid == 0) {
                __threadfence();
                const uint32_t prev = atomicAdd(P.tickets + c0, 1u);
                int todo = 0;                          // 1: merge this layer's row, 2: merge the row of the layer before
                if ((prev & ~kRequest) == (uint32_t)(n_parts - 1) && (layer == n_layers - 1 || (prev & kRequest))) todo |= 1;
                if (MAXL > 1 && layer > 0 && (prev & ~kRequest) == 0u) {
                    const uint32_t old = atomicOr(LS.layer[layer - 1].tickets + c0, kRequest);
                    if (old == (uint32_t)n_parts) todo |= 2;
                }
                *last_s = todo;
            }
            __syncthreads();
            const int todo = *last_s;
            if (todo) {
                __threadfence();
                const int first_slot = 2 * c0 + (row_start > partition_start(pt, cum, hkv, P.B, c0) ? 1 : 0);
                if constexpr (MAXL > 1) {
                    if (todo & 2) {
                        const DecodeParams& Q = LS.layer[layer - 1];
                        merge_row<D, NW * 32>(Q, first_slot, 2 * c0, n_parts, red, b, h);
                        if (tid == 0) Q.tickets[c0] = 0;
                    }
                }
                if (todo & 1) {
                    merge_row<D, NW * 32>(P, first_slot, 2 * c0, n_parts, red, b, h);
                    if (tid == 0) P.tickets[c0] = 0;
                }
            }
        }
        __syncthreads();
        pos += n_seg;
    }
    }   // layers
}

#include "decode_tmem.cuh"

// Per-device launch state of one kernel instantiation (dynamic shared memory opt-in, persistent grid size).
constexpr int kMaxDevices = 64;
struct LaunchCache {
    std::mutex mu;
    int grid[kMaxDevices] = {};
};

template <int D>
static int32_t run_tmem(mkv_pool* p, DecodeParams& prm, cudaStream_t s)
{
    using G = tm::TG<D>;
    auto kern = decode_tmem_kernel<D>;
    static LaunchCache cache;
    const int dev = p->device;
    if (dev < 0 || dev >= kMaxDevices) {
        set_last_error("decode attention: device index beyond the 64 this library keeps launch state for");
        return MKV_E_INVALID;
    }
    int grid;
    {
        std::lock_guard<std::mutex> lk(cache.mu);
        if (cache.grid[dev] == 0) {
            MKV_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM));
            cache.grid[dev] = p->dev.sm_count > kMaxCtas ? kMaxCtas : p->dev.sm_count;   // one block per SM: it takes all the tensor memory
        }
        grid = cache.grid[dev];
    }
    if (grid > prm.max_blocks) {
        set_last_error("decode attention: the scan launches more blocks on this GPU than the partial area has slots for");
        return MKV_E_INVALID;
    }
    kern<<<grid, tm::kThreads, G::SMEM, s>>>(prm);
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
}

template <int D, int NW, int NSTAGE, int MINB, bool SCORED, bool TILED, int MAXL, int FMT>
static int32_t run_tensor_fmt(mkv_pool* p, const LayerSet<MAXL>& ls, cudaStream_t s)
{
    using G = Geo<D, NW, NSTAGE, TILED>;
    auto kern = decode_tensor_kernel<D, NW, NSTAGE, MINB, SCORED, TILED, MAXL, FMT>;
    // pages of several tiles: one row of parked accumulators (8 D floats) per warp behind the usual layout
    constexpr int SMEM = G::SMEM + (TILED ? NW * 8 * D * 4 : 0);
    static_assert(SMEM <= 232448, "dynamic shared memory of one block");
    static LaunchCache cache;
    const int dev = p->device;
    if (dev < 0 || dev >= kMaxDevices) {
        set_last_error("decode attention: device index beyond the 64 this library keeps launch state for");
        return MKV_E_INVALID;
    }
    int grid;
    {
        std::lock_guard<std::mutex> lk(cache.mu);
        if (cache.grid[dev] == 0) {
            MKV_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM));
            int per_sm = 0;
            MKV_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, NW * 32, SMEM));
            if (per_sm < 1) return MKV_E_INVALID;
            const int g = p->dev.sm_count * per_sm;
            cache.grid[dev] = g > kMaxCtas ? kMaxCtas : g;
        }
        grid = cache.grid[dev];
    }
    if (grid > ls.layer[0].max_blocks) {
        set_last_error("decode attention: the scan launches more blocks on this GPU than the partial area has slots for");
        return MKV_E_INVALID;
    }
    kern<<<grid, NW * 32, SMEM, s>>>(ls);
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
}

// the pool's record format selects the instantiation
template <int D, int NW, int NSTAGE, int MINB, bool SCORED = false, bool TILED = false, int MAXL = 1>
static int32_t run_tensor(mkv_pool* p, const LayerSet<MAXL>& ls, cudaStream_t s)
{
    return p->fmt == 2 ? run_tensor_fmt<D, NW, NSTAGE, MINB, SCORED, TILED, MAXL, 2>(p, ls, s)
                       : run_tensor_fmt<D, NW, NSTAGE, MINB, SCORED, TILED, MAXL, 1>(p, ls, s);
}

template <int D, int NW, int NSTAGE, int MINB, bool SCORED = false, bool TILED = false>
static int32_t run_tensor1(mkv_pool* p, const DecodeParams& prm, cudaStream_t s)
{
    LayerSet<1> ls;
    ls.n = 1;
    ls.layer[0] = prm;
    return run_tensor<D, NW, NSTAGE, MINB, SCORED, TILED, 1>(p, ls, s);
}

int32_t launch_decode_tensor(mkv_pool* p, const void* q, const int32_t* bt, const uint8_t* tags,
                             const int32_t* lens, int B, int max_pages, float scale, float* out, float* lse,
                             void* ws, size_t, cudaStream_t s)
{
    // header: 256 reserved bytes, then kMaxCtas ticket words (cleared by mkv_workspace_init, left clear by every call)
    uint32_t* tickets = reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(ws) + 256);
    float* partials = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + decode_ws_header_bytes(B, p->hkv));
    return launch_decode_tensor_at(p, q, bt, tags, lens, B, max_pages, scale, out, lse, partials, tickets, kMaxCtas,
                                   nullptr, s);
}

int decode_tensor_partial_floats(int d) { return 8 * d + 16; }

// Second step of the scored variant: mass[b][hq][p] holds log2 of page p's exponential sum on an
// absolute origin; with the row's log-sum-exp it becomes q_p = 2^(that - lse2), and q~_p = q_p / sum q_p
// (Eq. score-global-weight and the normalisation over page-addressable mass that follows it).
// One block per (query head, request); entries beyond the request's pages are set to zero.
__global__ void __launch_bounds__(256) page_mass_finish_kernel(float* mass, const float* lse, const int32_t* lens,
                                                              int hq, int max_pages, int page_tokens)
{
    __shared__ float red[8];
    const int b = blockIdx.y, h = blockIdx.x, tid = threadIdx.x;
    const int len = lens[b], n_pages = len > 0 ? min((len + page_tokens - 1) / page_tokens, max_pages) : 0;
    float* row = mass + ((size_t)b * hq + h) * max_pages;
    const float lse2 = n_pages > 0 ? lse[(size_t)b * hq + h] * kLog2e : 0.f;
    float sum = 0.f;
    for (int p = tid; p < n_pages; p += 256) {
        const float qv = fast_exp2(row[p] - lse2);
        row[p] = qv;
        sum += qv;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if ((tid & 31) == 0) red[tid >> 5] = sum;
    __syncthreads();
    float total = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) total += red[w];
    const float inv = total > 0.f ? 1.f / total : 0.f;
    for (int p = tid; p < max_pages; p += 256) row[p] = p < n_pages ? row[p] * inv : 0.f;
}

// Eq. (attention-score): r_p = mean over the sampled heads of q~_{h,p}; a_p <- beta a_p + (1 - beta) r_p.
__global__ void __launch_bounds__(256) page_score_kernel(const float* mass, const int32_t* lens, int hq, int max_pages,
                                                         unsigned long long head_mask, float beta, float inv_heads,
                                                         float* score, int page_tokens)
{
    const int b = blockIdx.y, p = blockIdx.x * 256 + threadIdx.x;
    const int len = lens[b], n_pages = len > 0 ? min((len + page_tokens - 1) / page_tokens, max_pages) : 0;
    if (p >= n_pages) return;
    float r = 0.f;
    for (int h = 0; h < hq; ++h)
        if ((head_mask >> h) & 1ull) r += mass[((size_t)b * hq + h) * max_pages + p];
    float* a = score + (size_t)b * max_pages + p;
    *a = beta * *a + (1.f - beta) * (r * inv_heads);
}

// pages of several tiles: the scan adds parts of a page's sum to its entry, which therefore starts at -inf
__global__ void page_mass_clear_kernel(float* mass, size_t n)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) mass[i] = -CUDART_INF_F;
}

int32_t launch_page_mass_finish(float* mass, const float* lse, const int32_t* lens, int B, int hq, int max_pages,
                                int page_tokens, cudaStream_t s)
{
    page_mass_finish_kernel<<<dim3(hq, B), 256, 0, s>>>(mass, lse, lens, hq, max_pages, page_tokens);
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
}

int32_t launch_page_score(const float* mass, const int32_t* lens, int B, int hq, int max_pages, uint64_t head_mask,
                          float beta, float* score, int page_tokens, cudaStream_t s)
{
    int n = 0;
    for (int h = 0; h < hq; ++h) n += (int)((head_mask >> h) & 1ull);
    if (n == 0) return MKV_E_INVALID;
    page_score_kernel<<<dim3((max_pages + 255) / 256, B), 256, 0, s>>>(mass, lens, hq, max_pages, head_mask, beta,
                                                                         1.f / (float)n, score, page_tokens);
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
}

static DecodeParams make_params(mkv_pool* p, const void* q, const int32_t* bt, const uint8_t* tags, const int32_t* lens,
                                int B, int max_pages, float scale, float* out, float* lse, float* partials,
                                uint32_t* tickets, int max_blocks, float* mass)
{
    DecodeParams prm;
    prm.tiles = p->tiles;
    prm.fp8 = p->fp8; prm.tq3 = p->tq3;
    prm.fp8_pages = p->cfg.fp8_pages; prm.tq3_pages = p->cfg.tq3_pages;
    prm.hkv = p->hkv; prm.group = p->group;
    prm.k_scale = p->cfg.k_scale; prm.v_scale = p->cfg.v_scale;
    prm.sigma = p->sigma;
    prm.q = static_cast<const __nv_bfloat16*>(q);
    prm.bt = bt; prm.tags = tags; prm.lens = lens;
    prm.B = B; prm.max_pages = max_pages; prm.scale = scale;
    prm.out = out; prm.lse = lse;
    prm.partials = partials;
    prm.tickets = tickets;
    prm.max_blocks = max_blocks;
    prm.mass = mass;
    prm.status = p->status_dev;
    prm.wait_ns = p->wait_ns;
    return prm;
}

// Decode attention of several layers in one launch: layer i reads pool[i], q[i], bt[i], tags[i] and writes
// out[i], lse[i] (or none), with its own workspace ws[i]; the requests (lens, B, max_pages, scale) are common.
int32_t launch_decode_tensor_layers(mkv_pool* const* pools, const void* const* q, const int32_t* const* bt,
                                    const uint8_t* const* tags, const int32_t* lens, int B, int max_pages, float scale,
                                    float* const* out, float* const* lse, void* const* ws, int n_layers, cudaStream_t s)
{
    mkv_pool* p0 = pools[0];
    if (B > kMaxBatch || n_layers > kMaxLayers) return MKV_E_INVALID;
    if ((int64_t)max_pages * p0->tiles > 65535) {
        set_last_error("mkv_decode_attention_layers: more than 65535 16-token tiles per table row (1,048,560 tokens per request)");
        return MKV_E_INVALID;
    }
    LayerSet<kMaxLayers> ls;
    ls.n = n_layers;
    for (int i = 0; i < n_layers; ++i) {
        uint32_t* tickets = reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(ws[i]) + 256);
        float* partials = reinterpret_cast<float*>(static_cast<uint8_t*>(ws[i]) + decode_ws_header_bytes(B, p0->hkv));
        ls.layer[i] = make_params(pools[i], q[i], bt[i], tags[i], lens, B, max_pages, scale, out[i], lse ? lse[i] : nullptr,
                                  partials, tickets, kMaxCtas, nullptr);
    }
    if (p0->tiles > 1)                   // pages of several tiles (all pools of the call have the same page size)
        return p0->d == 128 ? run_tensor<128, 12, 4, 1, false, true, kMaxLayers>(p0, ls, s)
                            : run_tensor<256, 8, 4, 1, false, true, kMaxLayers>(p0, ls, s);
    return p0->d == 128 ? run_tensor<128, 12, 4, 1, false, false, kMaxLayers>(p0, ls, s)
                        : run_tensor<256, 8, 4, 1, false, false, kMaxLayers>(p0, ls, s);
}

int32_t launch_decode_tensor_at(mkv_pool* p, const void* q, const int32_t* bt, const uint8_t* tags,
                                const int32_t* lens, int B, int max_pages, float scale, float* out, float* lse,
                                float* partials, uint32_t* tickets, int max_blocks, float* mass, cudaStream_t s)
{
    if (B > kMaxBatch) return MKV_E_INVALID;
    if ((int64_t)max_pages * p->tiles > 65535) {   // the strided order multiplies two 16-token tile indices in 32 bits
        set_last_error("mkv_decode_attention: more than 65535 16-token tiles per table row (1,048,560 tokens per request)");
        return MKV_E_INVALID;
    }
    if (p->tiles > 1 && p->variant == MKV_DECODE_TMEM) {
        set_last_error("mkv_decode_attention: pages of several tiles are served by the tensor-core kernel");
        return MKV_E_INVALID;
    }
    if (p->fmt == 2 && p->variant == MKV_DECODE_TMEM) {
        set_last_error("mkv_decode_attention: record format 2 is served by the tensor-core and the CUDA-core kernels");
        return MKV_E_INVALID;
    }
    DecodeParams prm = make_params(p, q, bt, tags, lens, B, max_pages, scale, out, lse, partials, tickets, max_blocks, mass);
    if (mass) {                          // scored variant: the default launch shapes only
        int32_t rc;
        if (p->tiles > 1) {
            const size_t n = (size_t)B * p->hkv * p->group * max_pages;
            page_mass_clear_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(mass, n);
            MKV_CUDA(cudaGetLastError());
            rc = p->d == 128 ? run_tensor1<128, 12, 4, 1, true, true>(p, prm, s) : run_tensor1<256, 8, 4, 1, true, true>(p, prm, s);
        } else {
            rc = p->d == 128 ? run_tensor1<128, 12, 4, 1, true>(p, prm, s) : run_tensor1<256, 8, 4, 1, true>(p, prm, s);
        }
        if (rc != MKV_OK) return rc;
        return launch_page_mass_finish(mass, lse, lens, B, p->hkv * p->group, max_pages, p->cfg.page_size, s);
    }
    if (p->tiles > 1)                    // pages of several tiles: the default launch shapes only
        return p->d == 128 ? run_tensor1<128, 12, 4, 1, false, true>(p, prm, s) : run_tensor1<256, 8, 4, 1, false, true>(p, prm, s);
    if (p->variant == MKV_DECODE_TMEM && p->d == 256) return run_tmem<256>(p, prm, s);
    // launch shapes (warps per block, ring slots per warp, blocks per SM): 12 warps at 168 registers for
    // d = 128 (7 % faster than 16 warps at 128 registers), 8 warps for d = 256
    return p->d == 128 ? run_tensor1<128, 12, 4, 1>(p, prm, s) : run_tensor1<256, 8, 4, 1>(p, prm, s);
}

}  // namespace mkv
