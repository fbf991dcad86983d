// Decode attention with tcgen05 MMAs and tensor-memory accumulators (MKV_DECODE_TMEM), d = 256.
// Included by decode_tensor.cu (it shares that file's partition, unpack and merge code).
//
// Same one-pass mixed-format scan and the same split/merge as the mma.sync kernel; what changes is where
// the products run, who owns what, and that the stages of a page run in different warps at the same time.
// A block works on tiles of eight Stale pages (or four Recent/Anchor pages) = 128 tokens = the 128
// lanes of tensor memory.  Its 19 warps are seven groups, each a loop "wait for the inputs of my stage,
// do it, signal the outputs", coupled only by mbarriers (every wait bounded by wall time):
//   producer (1 warp)   bulk copies of a tile's records into one of four shared-memory tile buffers
//   key unpack (4)      each warp unpacks two pages into MMA A fragments exactly as the mma.sync kernel does
//                       and stores them to tensor memory (tcgen05.st.16x256b puts a fragment at rows g, g+8,
//                       32-bit columns 2tq, 2tq+1: a 16 x 16 tile with its K order permuted; the query tile
//                       in shared memory is written in the same permuted order)
//   score issue (1)     S[128 tokens x 16] = K q'^T: d/16 tcgen05.mma (M 128, N 16: the eight heads of the high
//                       half of the rotated query and of its low half), accumulating in tensor memory
//   softmax (4)         a thread owns one token (its tensor-memory lane): reads 16 scores, keeps the running
//                       maxima of the block, writes P (fp16 high | low halves) into the B tile of its page,
//                       page sums by shuffles over the 16 lanes of a page, rescale factors for the accumulators
//   value unpack (4)    per page each warp unpacks one quad of 16-channel blocks to tensor memory
//   value issue (1)     T[256 channels x 16] = codes^T P for two pages at a time (two 128-row halves each)
//   scale (4)           a thread owns two channels (its lane of the two halves): reads their results and applies
//                       the page's scale and zero in fp32 to 16 accumulators in registers -- two conversions per
//                       page and thread instead of the sixteen the fragment layout of mma.sync forces
// Key tiles, scores, value tiles and value products are double-buffered in tensor memory (480 of 512
// columns), so that all stages of consecutive tiles overlap.
namespace tm {

constexpr int kTile = 8;                            // Stale pages per tile (Recent/Anchor pages: half as many)
constexpr int kRing = 4;                            // tile buffers in shared memory
constexpr int kRoundT = 512;                        // positions whose table entries are listed at a time
constexpr int kWarps = 19;
constexpr int kThreads = kWarps * 32;
enum { kKU = 0, kSM = 4, kVU = 8, kSC = 12, kISS = 16, kISV = 17, kPR = 18 };   // first warp of every group
// tensor-memory columns
constexpr int kColK = 0;                            // key tile: d/2 columns (two fp16 per column)
constexpr int kColS = 128;                          // scores: 2 x 16 columns
constexpr int kColV = 160;                          // value tiles: 2 buffers x 2 pages x 2 halves x 8 columns
constexpr int kColT = 224;                          // value products: 4 buffers x 2 pages x 2 halves x 16 columns
constexpr int kTBuf = 4;
// mbarriers (index into the barrier array)
enum {
    kBarFull = 0,                                   // [kRing][kTile] records of a slot have landed (or the slot is unused)
    kBarTileFree = kRing * kTile,                   // [kRing] all 16 consumer warps are done with the buffer
    kBarKReady = kBarTileFree + kRing,              // [2] key tile stored (4 warps)
    kBarSFull = kBarKReady + 2,                     // [2] scores complete (commit); also: key tile may be overwritten
    kBarSFree = kBarSFull + 2,                      // [2] scores read (4 warps)
    kBarPReady = kBarSFree + 2,                     // [2] P tiles, page sums and rescale factors written (4 warps)
    kBarSCDone = kBarPReady + 2,                    // [2] scale warps are done with the tile (4 warps)
    kBarVReady = kBarSCDone + 2,                    // [2] value tiles of a batch stored (4 warps)
    kBarTFull = kBarVReady + 2,                     // [4] value products of a batch complete (commit); value tiles free
    kBarTFree = kBarTFull + 4,                      // [4] value products read (4 warps)
    kBarCount = kBarTFree + 4
};

template <int D>
struct TG {
    static constexpr int NB = D / 16;
    static constexpr int TQ3_REC = 16 * D + 32;
    static constexpr int FP8_HALF = 16 * D;
    static constexpr int SLOT = (TQ3_REC + 127) / 128 * 128;
    static constexpr int RING = kRing * kTile * SLOT;
    static constexpr int QTILES = NB * 512;                            // query B tiles: 16 rows x 16 k x 2 bytes per block
    static constexpr int OFF_QT = RING;                                // rotated query (rows 0-7 high, 8-15 low halves)
    static constexpr int OFF_QF = OFF_QT + QTILES;                     // plain query (rows 0-7; rows 8-15 zero)
    static constexpr int OFF_P = OFF_QF + QTILES;                      // 2 x kTile P tiles of 512 bytes (rows 0-7 high, 8-15 low)
    static constexpr int OFF_PS = OFF_P + 2 * kTile * 512;             // 2 x (page sums [kTile][8], rescale factors [8]) floats
    static constexpr int OFF_BAR = OFF_PS + 2 * (kTile + 1) * 32;
    static constexpr int OFF_LIST = OFF_BAR + ((kBarCount * 8 + 127) / 128) * 128;   // Stale ids, FP8 ids | valid << 27
    static constexpr int OFF_CNT = OFF_LIST + 2 * kRoundT * 4;         // n3, n8, 4 flags, 4 x 8 maxima
    static constexpr int OFF_CUM = OFF_CNT + 256;
    static constexpr int OFF_STRIDE = OFF_CUM + (kMaxBatch + 1) * 4;
    static constexpr int OFF_M = OFF_STRIDE + kMaxBatch * 4;
    static constexpr int OFF_L = OFF_M + 8 * 4;
    static constexpr int OFF_PART = OFF_L + 8 * 4;
    static constexpr int OFF_LAST = OFF_PART + ((int)sizeof(Partition) + 15) / 16 * 16;
    static constexpr int OFF_TMEM = OFF_LAST + 16;
    static constexpr int SMEM = OFF_TMEM + 16;
    static_assert(D == 256, "column map and channel ownership are laid out for d = 256");
    static_assert(RING >= 8 * D * 4 + kMaxCtas * 16 * 4 + 64, "ring doubles as reduction and merge buffer");
};

// ---- tcgen05 wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// one MMA A fragment (a0 .. a3 of m16k16) -> rows g, g+8 of the 16 lanes at taddr, 8 columns
__device__ __forceinline__ void tmem_st_frag(uint32_t taddr, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3)
{
    asm volatile("tcgen05.st.sync.aligned.16x256b.x1.b32 [%0], {%1,%2,%3,%4};" ::"r"(taddr), "r"(a0), "r"(a2), "r"(a1), "r"(a3) : "memory");
}
// four fragments (r[4w .. 4w+3] = a0, a2, a1, a3 of fragment w) -> 32 columns
__device__ __forceinline__ void tmem_st_frag4(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile("tcgen05.st.sync.aligned.16x256b.x4.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
                 "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
                 "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&r)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7]), "=f"(r[8]),
                   "=f"(r[9]), "=f"(r[10]), "=f"(r[11]), "=f"(r[12]), "=f"(r[13]), "=f"(r[14]), "=f"(r[15])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&r)[8])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7])
                 : "r"(taddr) : "memory");
}
// D[tmem] (+)= A[tmem] B[smem], kind f16, M and N from idesc
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
                 ::"r"(d), "r"(a), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// try_wait that lets the hardware suspend the thread (up to `ns`) until the phase completes, instead of spinning
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t ns)
{
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bar_sync(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void bar_arrive(int id, int count) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory"); }
// B tile in shared memory: 16 rows x 16 k of fp16, K-major, no swizzle: 8-row x 16-byte core matrices, the two
// K chunks 128 bytes apart, the two row groups 256 bytes apart
__device__ __forceinline__ uint64_t b_tile_desc(uint32_t saddr)
{
    return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)(128 >> 4) << 16) | ((uint64_t)(256 >> 4) << 32) | ((uint64_t)1 << 46);
}
__device__ __forceinline__ uint32_t b_tile_offset(int row, int k) { return (k >> 3) * 128 + (row >> 3) * 256 + (row & 7) * 16 + (k & 7) * 2; }
constexpr uint32_t kIdesc = (1u << 4) | (uint32_t)(16 >> 3) << 17 | (uint32_t)(128 >> 4) << 24;   // f16 x f16 -> f32, N 16, M 128

// position of a page's token in the K order of its value tile: Stale fragments hold tokens (2tq, 2tq+1) and
// (2tq+8, 2tq+9) in columns 2tq and 2tq+1; Recent/Anchor fragments (ldmatrix) tokens 4tq .. 4tq+3
__device__ __forceinline__ int k_of_token_tq3(int t) { return 4 * ((t & 7) >> 1) + (t & 1) + ((t >> 3) << 1); }


}  // namespace tm

template <int D>
__global__ void __launch_bounds__(tm::kThreads, 1) decode_tmem_kernel(const DecodeParams P)
{
    using namespace tm;
    using G = TG<D>;
    constexpr int NB = G::NB, NT = kThreads;
    constexpr uint32_t FULL = 0xffffffffu;
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    int* cum = reinterpret_cast<int*>(smem + G::OFF_CUM);
    int* strides = reinterpret_cast<int*>(smem + G::OFF_STRIDE);
    float* sm_m = reinterpret_cast<float*>(smem + G::OFF_M);
    float* sm_l = reinterpret_cast<float*>(smem + G::OFF_L);
    Partition* pt = reinterpret_cast<Partition*>(smem + G::OFF_PART);
    int* last_s = reinterpret_cast<int*>(smem + G::OFF_LAST);
    uint32_t* tmem_s = reinterpret_cast<uint32_t*>(smem + G::OFF_TMEM);
    float* red = reinterpret_cast<float*>(smem);            // [D][8] over the ring, between segments
    int* list3 = reinterpret_cast<int*>(smem + G::OFF_LIST);
    int* list8 = list3 + kRoundT;
    int* cnt = reinterpret_cast<int*>(smem + G::OFF_CNT);   // [0] n3, [1] n8, [4..7] flags, [8..39] maxima
    float* ps_all = reinterpret_cast<float*>(smem + G::OFF_PS);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    const int wq = warp & 3;                                 // tensor-memory subpartition of the warp (groups start at multiples of 4)
    const int hkv = P.hkv, GQ = P.group, hq = hkv * GQ;
    const uint32_t bars = sbase + G::OFF_BAR;
    auto bar = [&](int idx) -> uint32_t { return bars + 8 * idx; };

    // ---- prologue -------------------------------------------------------------------------------
    if (tid == 0) {
        for (int i = 0; i < kBarCount; ++i) {
            int count = 1;
            if (i >= kBarTileFree && i < kBarTileFree + kRing) count = 16;
            else if ((i >= kBarKReady && i < kBarSFull) || (i >= kBarSFree && i < kBarVReady + 2) || i >= kBarTFree) count = 4;
            mbar_init(bar(i), count);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int b = blockIdx.x; b < P.B; b += gridDim.x)
        if (P.lens[b] <= 0) {
            for (int i = tid; i < hq * D; i += NT) P.out[(size_t)b * hq * D + i] = 0.f;
            if (P.lse)
                for (int i = tid; i < hq; i += NT) P.lse[(size_t)b * hq + i] = -CUDART_INF_F;
        }
    // rows 8-15 of the plain query tiles stay zero for the whole launch
    for (int i = tid; i < G::QTILES / 4; i += NT) reinterpret_cast<uint32_t*>(smem + G::OFF_QF)[i] = 0;
    if (warp == 0) {
        int run = 0;
        for (int b0 = 0; b0 < P.B; b0 += 32) {
            const int b = b0 + lane;
            int n = 0;
            if (b < P.B) {
                int len = P.lens[b];
                if (len > P.max_pages * kPage) { atomicOr(P.status, kStBounds); len = P.max_pages * kPage; }   // a length beyond the table row is cut and flagged
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
        __syncwarp();
        build_partition(pt, cum, P.B, hkv, gridDim.x, lane);
    } else {
        for (int b = tid - 32; b < P.B; b += NT - 32) {
            const int len = min(max(P.lens[b], 0), P.max_pages * kPage), n = (len + kPage - 1) / kPage;
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
    if ((int)blockIdx.x >= pt->blocks) return;             // more blocks than work (nothing allocated yet)
    if (warp == kISS) tmem_alloc(smem_u32(tmem_s), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = *tmem_s;
    const uint32_t my_lanes = (uint32_t)(32 * wq) << 16;    // lanes of this warp's subpartition

    int my_start, my_end;
    partition_range(pt, cum, hkv, P.B, blockIdx.x, my_start, my_end);

    bool failed = false;
    const float sc2 = P.scale * kLog2e;
    uint32_t tcount = 0, bcount = 0;                         // tiles and value batches started so far (same in every warp)

    auto wait_bar = [&](int idx, uint32_t parity) {          // bounded; on time-out flag the pool and carry on
        const uint32_t a = bar(idx);
        if (failed || mbar_try_wait(a, parity)) return;
        // a waiting warp must not eat the issue slots of the working ones: poll, then sleep a little, and
        // look at the wall clock every 256 rounds
        unsigned long long t0 = 0, t1;
        for (int spins = 1;; ++spins) {
            if (mbar_try_wait(a, parity)) return;
            __nanosleep(spins < 4 ? 100 : 300);
            if ((spins & 255) == 0) {
                asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
                if (t0 == 0) t0 = t1;
                if (t1 - t0 > 20000000ull) {
                    failed = true;
                    atomicOr(P.status, kStTimeout);
                    return;
                }
            }
        }
    };
    // signal of a whole warp: its tensor-memory and shared-memory writes first, then one arrival
    auto warp_arrive = [&](int idx) {
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(idx));
    };
    auto wait_tile = [&](uint32_t t) {                       // all records of tile t are in its buffer
        const uint32_t rb = t % kRing, par = (t / kRing) & 1;
#pragma unroll 1
        for (int s = 0; s < kTile; ++s) wait_bar(kBarFull + rb * kTile + s, par);
    };

    int pos = my_start;
    int b = 0;
    while (pos < my_end) {
        while (cum[b + 1] <= pos) ++b;
        const int len = min(max(P.lens[b], 0), P.max_pages * kPage), n_pages = (len + kPage - 1) / kPage;
        const int h = (pos - cum[b]) / n_pages, pg0 = (pos - cum[b]) % n_pages;
        const int row_start = cum[b] + h * n_pages, row_end = row_start + n_pages;
        const int n_seg = min(my_end, row_end) - pos;
        const int32_t* bt_row = P.bt + (size_t)b * P.max_pages;
        const uint8_t* tag_row = P.tags + (size_t)b * P.max_pages;
        const int stride = strides[b];
        const int n_rounds = (n_seg + kRoundT - 1) / kRoundT;
        constexpr int EPL = D / 32;
        float qx[EPL];
#pragma unroll
        for (int r = 0; r < EPL; ++r)
            qx[r] = (warp < GQ) ? __bfloat162float(P.q[((size_t)b * hq + h * GQ + warp) * D + lane * EPL + r]) : 0.f;
        const uint8_t* tq3_base = P.tq3 + (size_t)h * G::TQ3_REC;
        const uint8_t* fp8_base = P.fp8 + (size_t)h * (2 * G::FP8_HALF);

        // softmax warps: running maxima of the eight heads (log2 units); scale warps: row sums and the accumulators
        // of channels (wq, lane) of the two 128-channel halves
        float m_run[8], l_run[8], acc0[8], acc1[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) { m_run[i] = -CUDART_INF_F; l_run[i] = 0.f; acc0[i] = 0.f; acc1[i] = 0.f; }

        // ---- query tiles (warps 0..7 rotate one head each), in the K order of the key fragments ---------
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
#pragma unroll
            for (int r = 0; r < EPL; ++r) {
                const int i = lane * EPL + r;
                {   // rotated query: dim 16 kb + dd sits at k = 4 ((dd & 7) >> 1) + 2 (dd >> 3) + (dd & 1) of block kb
                    const int kb = i >> 4, dd = i & 15, k = 4 * ((dd & 7) >> 1) + 2 * (dd >> 3) + (dd & 1);
                    const float v = a[r] * rs;
                    const __half vh = __float2half_rn(v);
                    *reinterpret_cast<__half*>(smem + G::OFF_QT + kb * 512 + b_tile_offset(hd, k)) = vh;
                    *reinterpret_cast<__half*>(smem + G::OFF_QT + kb * 512 + b_tile_offset(8 + hd, k)) =
                        __float2half_rn(v - __half2float(vh));
                }
                {   // plain query: dim 64 j + 16 t + 4 w + e sits at k = 4 t + e of block 4 j + w
                    const int j = i >> 6, t4 = (i & 63) >> 4, wv = (i & 15) >> 2, e = i & 3;
                    *reinterpret_cast<__half*>(smem + G::OFF_QF + (4 * j + wv) * 512 + b_tile_offset(hd, 4 * t4 + e)) =
                        __float2half_rn(qx[r]);
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }

        for (int round = 0; round < n_rounds; ++round) {
            // ---- table entries of the round -> two id lists (all warps) ----------------------------------
            if (tid == 0) { cnt[0] = 0; cnt[1] = 0; }
            __syncthreads();
            for (int i = round * kRoundT + tid; i < min(n_seg, (round + 1) * kRoundT); i += NT) {
                const int pg = (int)(((unsigned)(pg0 + i) * (unsigned)stride) % (unsigned)n_pages);
                const int id = bt_row[pg], tag = tag_row[pg], valid = min(kPage, len - pg * kPage);
                int kind = 0;
                if (tag == MKV_TAG_STALE) kind = (id >= 0 && id < P.tq3_pages && valid == kPage) ? 1 : 0;
                else kind = (tag <= MKV_TAG_ANCHOR && id >= 0 && id < P.fp8_pages) ? 2 : 0;
                if (kind == 1) list3[atomicAdd(&cnt[0], 1)] = id;
                else if (kind == 2) list8[atomicAdd(&cnt[1], 1)] = id | ((valid & 15) << 27);
                else atomicOr(P.status, kStBounds);     // never dereferenced
            }
            __syncthreads();                                 // lists (and, in the first round, the query tiles) complete
            const int n3 = cnt[0], n8 = cnt[1];
            const int tiles3 = (n3 + kTile - 1) / kTile, tiles8 = (n8 + kTile / 2 - 1) / (kTile / 2);
            const int n_tiles = tiles3 + tiles8;
            // tile ti of the round: format, first list entry, pages
            auto tile_info = [&](int ti, bool& stale, int& first, int& np) {
                stale = ti < tiles3;
                first = stale ? ti * kTile : (ti - tiles3) * (kTile / 2);
                np = stale ? min(kTile, n3 - first) : min(kTile / 2, n8 - first);
            };

            if (warp == kPR) {
                // ================= producer: records of a tile -> a tile buffer =================
                if (lane == 0) {
                    for (int ti = 0; ti < n_tiles; ++ti) {
                        bool stale; int first, np;
                        tile_info(ti, stale, first, np);
                        const uint32_t t = tcount + ti, rb = t % kRing;
                        if (t >= kRing) wait_bar(kBarTileFree + rb, ((t / kRing) - 1) & 1);
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        const uint32_t dst = sbase + rb * kTile * G::SLOT;
                        for (int s = 0; s < kTile; ++s) {
                            const uint32_t fb = bar(kBarFull + rb * kTile + s);
                            if (stale) {
                                if (s < np) {
                                    mbar_expect_tx(fb, G::TQ3_REC);
                                    bulk_load(dst + s * G::SLOT, tq3_base + (size_t)list3[first + s] * hkv * G::TQ3_REC, G::TQ3_REC, fb);
                                } else mbar_arrive(fb);
                            } else {
                                if ((s >> 1) < np) {
                                    const uint8_t* rec = fp8_base + (size_t)(list8[first + (s >> 1)] & 0x7FFFFFF) * hkv * (2 * G::FP8_HALF);
                                    mbar_expect_tx(fb, G::FP8_HALF);
                                    bulk_load(dst + s * G::SLOT, rec + (s & 1) * G::FP8_HALF, G::FP8_HALF, fb);
                                } else mbar_arrive(fb);
                            }
                        }
                    }
                }
                __syncwarp();
            } else if (warp == kISS) {
                // ================= score issue =================
                for (int ti = 0; ti < n_tiles; ++ti) {
                    bool stale; int first, np;
                    tile_info(ti, stale, first, np);
                    const uint32_t t = tcount + ti, kb2 = t & 1, par = (t >> 1) & 1;
                    wait_bar(kBarKReady + kb2, par);
                    if (t >= 2) wait_bar(kBarSFree + kb2, ((t >> 1) - 1) & 1);
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t qtile = sbase + (stale ? G::OFF_QT : G::OFF_QF);
#pragma unroll 1
                        for (int kb = 0; kb < NB; ++kb)
                            mma_ts(tb + kColS + 16 * kb2, tb + kColK + 8 * kb, b_tile_desc(qtile + kb * 512), kIdesc, kb > 0);
                        mma_commit(bar(kBarSFull + kb2));
                    }
                    __syncwarp();
                }
            } else if (warp == kISV) {
                // ================= value issue =================
                uint32_t bc = bcount;
                for (int ti = 0; ti < n_tiles; ++ti) {
                    bool stale; int first, np;
                    tile_info(ti, stale, first, np);
                    const uint32_t t = tcount + ti, pb = t & 1;
                    wait_bar(kBarPReady + pb, (t >> 1) & 1);
                    const int nb = (np + 1) / 2;
                    for (int bi = 0; bi < nb; ++bi, ++bc) {
                        const uint32_t vb = bc & 1, tbuf = bc % kTBuf;
                        wait_bar(kBarVReady + vb, (bc >> 1) & 1);
                        if (bc >= kTBuf) wait_bar(kBarTFree + tbuf, ((bc / kTBuf) - 1) & 1);
                        tc_fence_after();
                        if (lane == 0) {
#pragma unroll 1
                            for (int e = 0; e < 2; ++e) {
                                const int p = 2 * bi + e;
                                if (p >= np) break;
                                const uint64_t dp = b_tile_desc(sbase + G::OFF_P + (pb * kTile + p) * 512);
#pragma unroll
                                for (int m = 0; m < 2; ++m)
                                    mma_ts(tb + kColT + tbuf * 64 + e * 32 + m * 16, tb + kColV + vb * 32 + e * 16 + m * 8, dp, kIdesc, 0);
                            }
                            mma_commit(bar(kBarTFull + tbuf));
                        }
                        __syncwarp();
                    }
                }
            } else if (warp < kSM) {
                // ================= key unpack =================
                for (int ti = 0; ti < n_tiles; ++ti) {
                    bool stale; int first, np;
                    tile_info(ti, stale, first, np);
                    const uint32_t t = tcount + ti, rb = t % kRing, kb2 = t & 1;
                    const uint32_t tile = sbase + rb * kTile * G::SLOT;
                    wait_tile(t);
                    if (t >= 1) wait_bar(kBarSFull + ((t - 1) & 1), ((t - 1) >> 1) & 1);      // the score products of the tile before have read it
                    tc_fence_after();
#pragma unroll 1
                    for (int e = 0; e < 2; ++e) {
                        const int p = 2 * wq + e;
                        if (p >= np) continue;
                        const uint32_t dst = tb + kColK + my_lanes + ((uint32_t)(16 * e) << 16);
                        if (stale) {
                            const uint32_t sec = tile + p * G::SLOT + lane * 16;
#pragma unroll 1
                            for (int j = 0; j < NB / 4; ++j) {
                                // words 3j, 3j+1, 3j+2 of the lane (word i sits in chunk i / 4 at byte 4 (i % 4))
                                uint32_t A, Bw, Cw;
                                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(A) : "r"(sec + ((3 * j) >> 2) * 512 + ((3 * j) & 3) * 4));
                                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(Bw) : "r"(sec + ((3 * j + 1) >> 2) * 512 + ((3 * j + 1) & 3) * 4));
                                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(Cw) : "r"(sec + ((3 * j + 2) >> 2) * 512 + ((3 * j + 2) & 3) * 4));
                                uint32_t sel[4], r[16];
                                sel[0] = A & 0x77777777u;
                                sel[1] = Bw & 0x77777777u;
                                sel[2] = lop3_and_or(A >> 1, 0x44444444u, Cw & 0x33333333u);
                                sel[3] = lop3_and_or(Bw >> 1, 0x44444444u, (Cw >> 2) & 0x33333333u);
#pragma unroll
                                for (int w = 0; w < 4; ++w) {
                                    uint32_t a0, a1, a2, a3;
                                    key_lut4(sel[w], a0, a1);
                                    key_lut4(sel[w] >> 16, a2, a3);
                                    r[4 * w] = a0; r[4 * w + 1] = a2; r[4 * w + 2] = a1; r[4 * w + 3] = a3;
                                }
                                tmem_st_frag4(dst + 32 * j, r);
                            }
                        } else {
                            const uint32_t kaddr = tile + 2 * p * G::SLOT;
#pragma unroll 1
                            for (int j = 0; j < D / 64; ++j) {
                                const uint4 r0 = lds128(kaddr + g * D + 64 * j + 16 * tq);
                                const uint4 r1 = lds128(kaddr + (g + 8) * D + 64 * j + 16 * tq);
                                const uint32_t w0[4] = {r0.x, r0.y, r0.z, r0.w}, w1[4] = {r1.x, r1.y, r1.z, r1.w};
                                uint32_t r[16];
#pragma unroll
                                for (int w = 0; w < 4; ++w) {
                                    r[4 * w] = e4m3x2_to_f16x2((uint16_t)(w0[w] & 0xFFFFu));
                                    r[4 * w + 1] = e4m3x2_to_f16x2((uint16_t)(w0[w] >> 16));
                                    r[4 * w + 2] = e4m3x2_to_f16x2((uint16_t)(w1[w] & 0xFFFFu));
                                    r[4 * w + 3] = e4m3x2_to_f16x2((uint16_t)(w1[w] >> 16));
                                }
                                tmem_st_frag4(dst + 32 * j, r);
                            }
                        }
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    warp_arrive(kBarKReady + kb2);
                    warp_arrive(kBarTileFree + rb);
                }
            } else if (warp < kVU) {
                // ================= softmax =================
                for (int ti = 0; ti < n_tiles; ++ti) {
                    bool stale; int first, np;
                    tile_info(ti, stale, first, np);
                    const uint32_t t = tcount + ti, rb = t % kRing, sb = t & 1, par = (t >> 1) & 1;
                    const uint32_t tile = sbase + rb * kTile * G::SLOT;
                    const int p_me = 2 * wq + (lane >> 4), tok = lane & 15;
                    int valid = kPage;
                    if (!stale && p_me < np) { const int v = (list8[first + p_me] >> 27) & 15; valid = v ? v : kPage; }
                    const bool live = p_me < np && tok < valid;
                    wait_tile(t);
                    float rsc = sc2 * P.k_scale;
                    if (stale) rsc = __half2float(__ushort_as_half(lds16(tile + (p_me < np ? p_me : 0) * G::SLOT + 12 * D + 2 * tok))) * sc2;
                    warp_arrive(kBarTileFree + rb);
                    wait_bar(kBarSFull + sb, par);
                    tc_fence_after();
                    float s[8];
                    {
                        float c[16];
                        tmem_ld16(tb + kColS + 16 * sb + my_lanes, c);
                        tmem_wait_ld();
                        tc_fence_before();
                        warp_arrive(kBarSFree + sb);
#pragma unroll
                        for (int i = 0; i < 8; ++i) s[i] = live ? (c[i] + c[8 + i]) * rsc : -CUDART_INF_F;
                    }
                    // running maxima: raised only when some score of the tile exceeds them by 2^kRescaleSlack
                    float fs[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) fs[i] = 1.f;
                    bool ex = false;
#pragma unroll
                    for (int i = 0; i < 8; ++i) ex = ex || (s[i] > m_run[i] + kRescaleSlack);
                    ex = __any_sync(FULL, ex);
                    if (lane == 0) cnt[4 + wq] = ex ? 1 : 0;
                    bar_sync(1, 128);
                    if (cnt[4] | cnt[5] | cnt[6] | cnt[7]) {
                        float mx[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            float v = s[i];
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(FULL, v, o));
                            mx[i] = v;
                        }
                        if (lane < 8) {
                            float v = mx[0];
#pragma unroll
                            for (int i = 1; i < 8; ++i) v = lane == i ? mx[i] : v;
                            reinterpret_cast<float*>(cnt)[8 + wq * 8 + lane] = v;
                        }
                        bar_sync(1, 128);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float* q4 = reinterpret_cast<const float*>(cnt) + 8 + i;
                            const float nm = fmaxf(fmaxf(q4[0], q4[8]), fmaxf(q4[16], q4[24]));
                            if (nm > m_run[i] + kRescaleSlack) {
                                fs[i] = m_run[i] == -CUDART_INF_F ? 0.f : fast_exp2(m_run[i] - nm);
                                m_run[i] = nm;
                            }
                        }
                    }
                    bar_sync(1, 128);                        // flags and maxima are read; they may be rewritten for the next tile
                    // the tile's P tiles, page sums and rescale factors go to set sb once the scale warps are done with it
                    if (t >= 2) wait_bar(kBarSCDone + sb, ((t >> 1) - 1) & 1);
                    float* ps_s = ps_all + sb * (kTile + 1) * 8;
                    {
                        const int kk = stale ? k_of_token_tq3(tok) : tok;
                        const uint32_t tp = sbase + G::OFF_P + (sb * kTile + (p_me & (kTile - 1))) * 512;
                        float pv[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float pr = fast_exp2(s[i] - m_run[i]);      // exp2(-inf) = 0 for dead rows
                            const __half ph = __float2half_rn(pr);
                            const __half pl = __float2half_rn(pr - __half2float(ph));
                            if (p_me < np) {
                                asm volatile("st.shared.u16 [%0], %1;" ::"r"(tp + b_tile_offset(i, kk)), "h"(__half_as_ushort(ph)) : "memory");
                                asm volatile("st.shared.u16 [%0], %1;" ::"r"(tp + b_tile_offset(8 + i, kk)), "h"(__half_as_ushort(pl)) : "memory");
                            }
                            pv[i] = __half2float(ph) + __half2float(pl);
                        }
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
#pragma unroll
                            for (int o = 8; o > 0; o >>= 1) pv[i] += __shfl_xor_sync(FULL, pv[i], o);
                        }
                        if (tok == 0) {
                            *reinterpret_cast<float4*>(ps_s + p_me * 8) = make_float4(pv[0], pv[1], pv[2], pv[3]);
                            *reinterpret_cast<float4*>(ps_s + p_me * 8 + 4) = make_float4(pv[4], pv[5], pv[6], pv[7]);
                        }
                        if (warp == kSM && lane == 0) {
                            *reinterpret_cast<float4*>(ps_s + kTile * 8) = make_float4(fs[0], fs[1], fs[2], fs[3]);
                            *reinterpret_cast<float4*>(ps_s + kTile * 8 + 4) = make_float4(fs[4], fs[5], fs[6], fs[7]);
                        }
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    }
                    warp_arrive(kBarPReady + sb);
                }
            } else if (warp < kSC) {
                // ================= value unpack =================
                uint32_t bc = bcount;
                for (int ti = 0; ti < n_tiles; ++ti) {
                    bool stale; int first, np;
                    tile_info(ti, stale, first, np);
                    const uint32_t t = tcount + ti, rb = t % kRing;
                    const uint32_t tile = sbase + rb * kTile * G::SLOT;
                    wait_tile(t);
                    const int nb = (np + 1) / 2;
                    for (int bi = 0; bi < nb; ++bi, ++bc) {
                        const uint32_t vb = bc & 1;
                        if (bc >= 2) wait_bar(kBarTFull + (bc - 2) % kTBuf, ((bc - 2) / kTBuf) & 1);     // the products of the batch before last have read it
                        tc_fence_after();
#pragma unroll 1
                        for (int e = 0; e < 2; ++e) {
                            const int p = 2 * bi + e;
                            if (p >= np) break;
                            const uint32_t dV = tb + kColV + vb * 32 + e * 16 + my_lanes;   // half m at + 8 m, rows 16..31 at + (16 << 16)
                            if (stale) {
                                const uint32_t sec = tile + p * G::SLOT + 6 * D;
                                uint32_t W[3];
#pragma unroll
                                for (int k = 0; k < 3; ++k) {
                                    const int i = 3 * wq + k;
                                    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(W[k]) : "r"(sec + (i >> 2) * 512 + lane * 16 + (i & 3) * 4));
                                }
                                const uint32_t X1 = prmt(W[0], W[1], 0x6341u), X0 = prmt(W[1], W[2], 0x6341u), X2 = W[2] >> 8;
                                tmem_st_frag(dV, value_code<0>(W[0]), value_code<3>(W[0]), value_code<6>(W[0]), value_code<1>(X1));
                                tmem_st_frag(dV + (16u << 16), value_code<4>(X1), value_code<7>(X1), value_code<2>(W[1]), value_code<5>(W[1]));
                                tmem_st_frag(dV + 8, value_code<0>(X0), value_code<3>(X0), value_code<6>(X0), value_code<1>(W[2]));
                                tmem_st_frag(dV + 8 + (16u << 16), value_code<4>(W[2]), value_code<7>(W[2]), value_code<2>(X2), value_code<5>(X2));
                            } else {
                                const uint32_t vaddr = tile + (2 * p + 1) * G::SLOT;
                                const int v = (list8[first + p] >> 27) & 15, nv = v ? v : kPage;
                                const uint32_t keep = (4 * tq < nv ? 0x000000FFu : 0u) | (4 * tq + 1 < nv ? 0x0000FF00u : 0u) |
                                                      (4 * tq + 2 < nv ? 0x00FF0000u : 0u) | (4 * tq + 3 < nv ? 0xFF000000u : 0u);
#pragma unroll
                                for (int m = 0; m < 2; ++m) {
                                    uint32_t v4[4];
                                    ldmatrix_x4(vaddr + (4 * wq + 2 * m) * 256 + lane * 16, v4[0], v4[1], v4[2], v4[3]);
#pragma unroll
                                    for (int k = 0; k < 2; ++k) {
                                        const uint32_t lo = v4[2 * k] & keep, hi = v4[2 * k + 1] & keep;
                                        tmem_st_frag(dV + 8 * m + ((uint32_t)(16 * k) << 16), e4m3x2_to_f16x2((uint16_t)(lo & 0xFFFFu)),
                                                     e4m3x2_to_f16x2((uint16_t)(hi & 0xFFFFu)), e4m3x2_to_f16x2((uint16_t)(lo >> 16)),
                                                     e4m3x2_to_f16x2((uint16_t)(hi >> 16)));
                                    }
                                }
                            }
                        }
                        tmem_wait_st();
                        tc_fence_before();
                        warp_arrive(kBarVReady + vb);
                    }
                    warp_arrive(kBarTileFree + rb);
                }
            } else {
                // ================= scale =================
                uint32_t bc = bcount;
                for (int ti = 0; ti < n_tiles; ++ti) {
                    bool stale; int first, np;
                    tile_info(ti, stale, first, np);
                    const uint32_t t = tcount + ti, rb = t % kRing, pb = t & 1;
                    const uint32_t tile = sbase + rb * kTile * G::SLOT;
                    const float* ps_s = ps_all + pb * (kTile + 1) * 8;
                    wait_tile(t);
                    wait_bar(kBarPReady + pb, (t >> 1) & 1);
                    {
                        const float4 fa = *reinterpret_cast<const float4*>(ps_s + kTile * 8), fb = *reinterpret_cast<const float4*>(ps_s + kTile * 8 + 4);
                        const float fsc[8] = {fa.x, fa.y, fa.z, fa.w, fb.x, fb.y, fb.z, fb.w};
#pragma unroll
                        for (int i = 0; i < 8; ++i) { l_run[i] *= fsc[i]; acc0[i] *= fsc[i]; acc1[i] *= fsc[i]; }
                    }
                    const int nb = (np + 1) / 2;
                    for (int bi = 0; bi < nb; ++bi, ++bc) {
                        const uint32_t vb = bc % kTBuf;
                        wait_bar(kBarTFull + vb, (bc / kTBuf) & 1);
                        tc_fence_after();
                        const int pn = min(2, np - 2 * bi);
#pragma unroll 1
                        for (int e = 0; e < pn; ++e) {
                            float t0[16], t1[16];
                            tmem_ld16(tb + kColT + vb * 64 + e * 32 + my_lanes, t0);
                            tmem_ld16(tb + kColT + vb * 64 + e * 32 + 16 + my_lanes, t1);
                            tmem_wait_ld();
                            if (e == pn - 1) {
                                tc_fence_before();
                                warp_arrive(kBarTFree + vb);
                            }
                            const int p = 2 * bi + e;
                            const float4 pa = *reinterpret_cast<const float4*>(ps_s + p * 8), pbv = *reinterpret_cast<const float4*>(ps_s + p * 8 + 4);
                            const float ps[8] = {pa.x, pa.y, pa.z, pa.w, pbv.x, pbv.y, pbv.z, pbv.w};
                            float sc0 = P.v_scale, zp0 = 0.f, sc1 = P.v_scale, zp1 = 0.f;
                            if (stale) {
                                // channel 16 cb + row: halves (scale, zero) at ((cb/2) 64 + (row%8) 8 + 4 (cb%2) + row/8) and + 2
                                const uint32_t meta = tile + p * G::SLOT + 12 * D + 32;
                                const int row = lane & 15, cb0 = 4 * wq + (lane >> 4), cb1 = cb0 + 2;
                                const uint32_t i0 = (cb0 >> 1) * 64 + (row & 7) * 8 + 4 * (cb0 & 1) + (row >> 3);
                                const uint32_t i1 = (cb1 >> 1) * 64 + (row & 7) * 8 + 4 * (cb1 & 1) + (row >> 3);
                                sc0 = __half2float(__ushort_as_half(lds16(meta + 2 * i0)));
                                zp0 = __half2float(__ushort_as_half(lds16(meta + 2 * i0 + 4)));
                                sc1 = __half2float(__ushort_as_half(lds16(meta + 2 * i1)));
                                zp1 = __half2float(__ushort_as_half(lds16(meta + 2 * i1 + 4)));
                            }
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                acc0[i] = fmaf(sc0, t0[i] + t0[8 + i], fmaf(zp0, ps[i], acc0[i]));
                                acc1[i] = fmaf(sc1, t1[i] + t1[8 + i], fmaf(zp1, ps[i], acc1[i]));
                                l_run[i] += ps[i];
                            }
                        }
                    }
                    warp_arrive(kBarTileFree + rb);
                    warp_arrive(kBarSCDone + pb);
                }
            }
            // every warp advances the counters by what the round held
            for (int ti = 0; ti < n_tiles; ++ti) {
                bool stale; int first, np;
                tile_info(ti, stale, first, np);
                bcount += (np + 1) / 2;
            }
            tcount += n_tiles;
            failed = __any_sync(FULL, failed);
        }

        // ---- results of the row (ring memory is idle now) ------------------------------------------------
        tc_fence_before();
        __syncthreads();
        if (warp == kSM && lane == 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i) sm_m[i] = m_run[i];
        }
        if (warp >= kSC && warp < kISS) {
            const int c0 = 16 * (4 * wq + (lane >> 4)) + (lane & 15), c1 = c0 + 32;
            *reinterpret_cast<float4*>(red + c0 * 8) = make_float4(acc0[0], acc0[1], acc0[2], acc0[3]);
            *reinterpret_cast<float4*>(red + c0 * 8 + 4) = make_float4(acc0[4], acc0[5], acc0[6], acc0[7]);
            *reinterpret_cast<float4*>(red + c1 * 8) = make_float4(acc1[0], acc1[1], acc1[2], acc1[3]);
            *reinterpret_cast<float4*>(red + c1 * 8 + 4) = make_float4(acc1[4], acc1[5], acc1[6], acc1[7]);
            if (warp == kSC && lane == 0) {
#pragma unroll
                for (int i = 0; i < 8; ++i) sm_l[i] = l_run[i];
            }
        }
        __syncthreads();

        const bool whole_row = (pos == row_start) && (pos + n_seg == row_end);
        if (whole_row) {
            for (int e = tid; e < 8 * D; e += NT) {
                const int head = e & 7, ch = e >> 3;
                if (head >= GQ) continue;
                const float l = sm_l[head];
                P.out[((size_t)b * hq + h * GQ + head) * D + ch] = l > 0.f ? red[e] / l : 0.f;
            }
            if (P.lse && tid < GQ)
                P.lse[(size_t)b * hq + h * GQ + tid] = sm_l[tid] > 0.f ? (sm_m[tid] + log2f(sm_l[tid])) * kLn2 : -CUDART_INF_F;
        } else {
            float* slot = P.partials + (size_t)(2 * blockIdx.x + (pos != my_start ? 1 : 0)) * (8 * D + 16);
            for (int e = tid; e < 8 * D; e += NT) slot[e] = red[e];
            if (tid < 8) {
                slot[8 * D + tid] = sm_m[tid];
                slot[8 * D + 8 + tid] = sm_l[tid];
            }
            int c0, c1;
            partition_blocks_of_row(pt, cum, P.B, b * hkv + h, row_start, row_end, c0, c1);
            const int n_parts = c1 - c0 + 1;
            __syncthreads();
            if (tid == 0) {
                __threadfence();
                const uint32_t prev = atomicAdd(P.tickets + c0, 1u);
                const int last = prev == (uint32_t)(n_parts - 1);
                if (last) P.tickets[c0] = 0;
                *last_s = last;
            }
            __syncthreads();
            if (*last_s) {
                __threadfence();
                const int first_slot = 2 * c0 + (row_start > partition_start(pt, cum, hkv, P.B, c0) ? 1 : 0);
                merge_row<D, NT, 16>(P, first_slot, 2 * c0, n_parts, red, b, h);
            }
        }
        __syncthreads();
        pos += n_seg;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kISS) tmem_dealloc(tb, 512);
}
