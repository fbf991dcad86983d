// Decode attention with tcgen05 MMAs and tensor-memory accumulators (MKV_DECODE_TMEM), d = 256.
// Included by decode_tensor.cu (it shares that file's partition, unpack and merge code).
//
// Same one-pass mixed-format scan and the same split/merge as the mma.sync kernel; what changes is where
// the products run and who owns what:
//   * a block holds two teams of four worker warps plus one issuing warp per team.  A team works on a
//     tile of eight Stale pages (or four Recent/Anchor pages) of its share of the row at a time.
//   * keys: every worker warp unpacks two pages into MMA A fragments exactly as the mma.sync kernel
//     does, but stores them to tensor memory (tcgen05.st.16x256b puts a fragment's registers at
//     (row g | g+8, 32-bit columns 2tq, 2tq+1), i.e. a 16 x 16 tile with its K order permuted; the
//     query tile in shared memory is written in the same permuted order).  One thread of the issuing
//     warp then runs S[128 tokens x 16] = K q'^T as d/16 tcgen05.mma (M 128, N 16: eight heads of the
//     high half of the rotated query and eight of the low half), accumulating in tensor memory.
//   * softmax: a worker thread owns one token (tensor-memory lane = token): it reads its 16 scores,
//     forms P for the eight heads and writes P (fp16 high and low halves) into the B tiles of the
//     value product; page sums come from shuffles over the 16 lanes of a page.
//   * values: for every page the four worker warps unpack one quad of 16-channel blocks each into
//     tensor memory; T[256 channels x 8 heads] = codes^T P runs as four tcgen05.mma (two 128-row
//     halves x {P high, P low}).  A worker thread owns two channels (its lane of the two halves): it
//     reads their 2 x 8 results and applies the page's scale and zero in fp32 to 16 accumulators in
//     registers -- two conversions per page and thread instead of the sixteen the fragment layout
//     of mma.sync forces, and no accumulator fragments in registers.
//   * hand-over between workers and the issuing warp is by named barriers (workers arrive, the
//     issuing warp waits) and by mbarriers signalled with tcgen05.commit (workers wait, bounded by wall
//     time like every other wait here); worker warps never wait for each other inside a page.
namespace tm {

constexpr int kTeams = 2;                           // teams per block
constexpr int kTile = 8;                            // Stale pages per tile (Recent/Anchor pages: half as many)
constexpr int kRoundT = 256;                        // positions of a team whose table entries are listed at a time
constexpr int kWorkerWarps = kTeams * 4;            // warps 0 .. 7; warps 8, 9 issue the MMAs of team 0, 1
constexpr int kThreads = (kWorkerWarps + kTeams) * 32;
constexpr int kTeamCols = 256;                      // tensor-memory columns of a team
// columns inside a team's range
constexpr int kColK = 0;                            // key tile: d/2 columns (two fp16 per column)
constexpr int kColS = 128;                          // scores: 16 columns
constexpr int kColV = 144;                          // value tiles: 2 buffers x 2 pages x 2 halves x 8 columns
constexpr int kColT = 0;                            // value products: 2 buffers x 2 pages x 2 halves x 16 columns, over the key
                                                    // tile (dead once the scores are complete; every warp touches its own lanes only)

template <int D>
struct TG {
    static constexpr int NB = D / 16;
    static constexpr int TQ3_REC = 16 * D + 32;
    static constexpr int FP8_HALF = 16 * D;
    static constexpr int SLOT = (TQ3_REC + 127) / 128 * 128;
    static constexpr int RING = kTeams * 2 * kTile * SLOT;             // per team two buffers of eight slots
    static constexpr int QTILES = NB * 512;                            // query B tiles: 16 rows x 16 k x 2 bytes per block
    static constexpr int OFF_QT = RING;                                // rotated query (rows 0-7 high, 8-15 low halves)
    static constexpr int OFF_QF = OFF_QT + QTILES;                     // plain query (rows 0-7; rows 8-15 zero)
    static constexpr int OFF_P = OFF_QF + QTILES;                      // per team: kTile P tiles of 512 bytes (rows 0-7 high, 8-15 low halves)
    static constexpr int OFF_PS = OFF_P + kTeams * kTile * 512;        // per team: page sums [kTile][8] floats
    static constexpr int OFF_BAR = OFF_PS + kTeams * kTile * 32;       // per team: 16 slot barriers, S, T0, T1 (32 x 8 bytes)
    static constexpr int OFF_LIST = OFF_BAR + kTeams * 256;            // per team: Stale ids, FP8 ids | valid << 27
    static constexpr int OFF_CNT = OFF_LIST + kTeams * 2 * kRoundT * 4;    // per team: n3, n8, 4 flags, 4 x 8 maxima
    static constexpr int OFF_CUM = OFF_CNT + kTeams * 256;
    static constexpr int OFF_STRIDE = OFF_CUM + (kMaxBatch + 1) * 4;
    static constexpr int OFF_M = OFF_STRIDE + kMaxBatch * 4;
    static constexpr int OFF_L = OFF_M + kTeams * 8 * 4;
    static constexpr int OFF_PART = OFF_L + kTeams * 8 * 4;
    static constexpr int OFF_LAST = OFF_PART + ((int)sizeof(Partition) + 15) / 16 * 16;
    static constexpr int OFF_TMEM = OFF_LAST + 16;
    static constexpr int SMEM = OFF_TMEM + 16;
    static_assert(D == 256, "column map and channel ownership are laid out for d = 256");
    static_assert(RING >= kTeams * 8 * D * 4 + kMaxCtas * 16 * 4 + 64, "ring doubles as reduction and merge buffer");
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
    constexpr int NB = G::NB, NT = kThreads, NU = kTeams, LW = 3 * NB / 4;
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
    float* red = reinterpret_cast<float*>(smem);            // [teams][D][8] over the ring, between segments

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    const bool worker = warp < kWorkerWarps;
    const int team = worker ? warp >> 2 : warp - kWorkerWarps;
    const int wq = warp & 3;                                 // worker: tensor-memory subpartition = quad of value blocks
    const int ttid = (warp & 3) * 32 + lane;                 // worker: thread index inside the team
    const int hkv = P.hkv, GQ = P.group, hq = hkv * GQ;
    // named barriers of the team: workers only; key tile ready; value tile ready (two, alternating); round hand-over
    const int idW = 1 + 5 * team, idK = 2 + 5 * team, idK2 = 3 + 5 * team, idV0 = 4 + 5 * team, idR = 11 + team;

    // ---- prologue -------------------------------------------------------------------------------
    if (tid == 0) {
        for (int i = 0; i < kTeams * 32; ++i) mbar_init(sbase + G::OFF_BAR + 8 * i, 1);
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
        __syncwarp();
        build_partition(pt, cum, P.lens, P.B, hkv, gridDim.x, lane);
    } else {
        for (int b = tid - 32; b < P.B; b += NT - 32) {
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
    if ((int)blockIdx.x >= pt->blocks) return;             // more blocks than work (nothing allocated yet)
    if (warp == kWorkerWarps) tmem_alloc(smem_u32(tmem_s), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_all = *tmem_s;
    const uint32_t tb = tmem_all + team * kTeamCols;        // this team's columns (lane field zero)
    const uint32_t my_lanes = (uint32_t)(32 * wq) << 16;    // worker: lanes of its subpartition

    int my_start, my_end;
    partition_range(pt, cum, hkv, P.B, blockIdx.x, my_start, my_end);

    bool failed = false;
    const uint32_t bars = sbase + G::OFF_BAR + team * 256;  // slot barriers 0..15, S = 16, T0 = 17, T1 = 18
    const uint32_t ring = sbase + team * 2 * kTile * G::SLOT;
    const uint32_t ptiles = sbase + G::OFF_P + team * kTile * 512;
    float* ps_s = reinterpret_cast<float*>(smem + G::OFF_PS) + team * kTile * 8;
    int* list3 = reinterpret_cast<int*>(smem + G::OFF_LIST) + team * 2 * kRoundT;
    int* list8 = list3 + kRoundT;
    int* cnt = reinterpret_cast<int*>(smem + G::OFF_CNT) + team * 64;      // [0] n3, [1] n8, [4..7] flags, [8..39] maxima
    const float sc2 = P.scale * kLog2e;
    uint32_t tcount = 0, scount = 0, tcnt0 = 0, tcnt1 = 0;   // tiles started, S and T completions waited for

    auto wait_bar = [&](uint32_t bar, uint32_t parity) {     // bounded; on time-out flag the pool and carry on
        if (failed || mbar_try_wait(bar, parity)) return;
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
    };

#ifdef MKV_TIMELINE
    unsigned long long tl_acc[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}, tl_last = tl_now(), tl_begin = tl_last;
#define TM_STAMP(k) do { if (tid == 0) { const unsigned long long t__ = tl_now(); tl_acc[k] += t__ - tl_last; tl_last = t__; } } while (0)
#else
#define TM_STAMP(k)
#endif
    int pos = my_start;
    int b = 0;
    while (pos < my_end) {
        while (cum[b + 1] <= pos) ++b;
        const int len = P.lens[b], n_pages = (len + kPage - 1) / kPage;
        const int h = (pos - cum[b]) / n_pages, pg0 = (pos - cum[b]) % n_pages;
        const int row_start = cum[b] + h * n_pages, row_end = row_start + n_pages;
        const int n_seg = min(my_end, row_end) - pos;
        const int32_t* bt_row = P.bt + (size_t)b * P.max_pages;
        const uint8_t* tag_row = P.tags + (size_t)b * P.max_pages;
        const int stride = strides[b];
        const int team_first = (int)(((unsigned)n_seg * (unsigned)team) / kTeams);
        const int n_team = (int)(((unsigned)n_seg * (unsigned)(team + 1)) / kTeams) - team_first;
        const int n_rounds = (n_team + kRoundT - 1) / kRoundT;
        constexpr int EPL = D / 32;
        float qx[EPL];
#pragma unroll
        for (int r = 0; r < EPL; ++r)
            qx[r] = (warp < GQ) ? __bfloat162float(P.q[((size_t)b * hq + h * GQ + warp) * D + lane * EPL + r]) : 0.f;
        const uint8_t* tq3_base = P.tq3 + (size_t)h * G::TQ3_REC;
        const uint8_t* fp8_base = P.fp8 + (size_t)h * (2 * G::FP8_HALF);

        // state of the team for this row (the same in all its worker threads): running maxima and row sums of
        // the eight heads in log2 units; a worker thread's accumulators: channels (wq, lane) of the two halves
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
        __syncthreads();
        TM_STAMP(1);

        for (int round = 0; round < n_rounds; ++round) {
            // ---- table entries of the round -> two id lists of the team ---------------------------------
            if (worker) {
                if (ttid == 0) { cnt[0] = 0; cnt[1] = 0; }
                bar_sync(idW, 128);
#pragma unroll 1
                for (int k = 0; k < kRoundT / 128; ++k) {
                    const int i = round * kRoundT + k * 128 + ttid;
                    if (i < n_team) {
                        const int pg = (int)(((unsigned)(pg0 + team_first + i) * (unsigned)stride) % (unsigned)n_pages);
                        const int id = bt_row[pg], tag = tag_row[pg], valid = min(kPage, len - pg * kPage);
                        int kind = 0;
                        if (tag == MKV_TAG_STALE) kind = (id >= 0 && id < P.tq3_pages && valid == kPage) ? 1 : 0;
                        else kind = (tag <= MKV_TAG_ANCHOR && id >= 0 && id < P.fp8_pages) ? 2 : 0;
                        if (kind == 1) list3[atomicAdd(&cnt[0], 1)] = id;
                        else if (kind == 2) list8[atomicAdd(&cnt[1], 1)] = id | ((valid & 15) << 27);
                        else atomicOr(P.status, kStBounds);     // never dereferenced
                    }
                }
            }
            bar_sync(idR, 160);                              // lists complete (workers and the issuing warp)
            const int n3 = cnt[0], n8 = cnt[1];
            const int tiles3 = (n3 + kTile - 1) / kTile, tiles8 = (n8 + kTile / 2 - 1) / (kTile / 2);
            const int n_tiles = tiles3 + tiles8;

            // copies of tile ti into buffer `buf`: worker warp wq owns slots 2wq, 2wq + 1 (a Stale page each, or
            // the key and the value half of one Recent/Anchor page); unused slots just complete their phase
            auto issue_tile = [&](int ti, uint32_t buf) {
                if (lane != 0) return;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                const uint32_t s0 = 2 * wq, dst = ring + (buf * kTile + s0) * G::SLOT, bar0 = bars + 8 * (buf * kTile + s0);
                if (ti < tiles3) {
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int i = ti * kTile + s0 + e;
                        if (i < n3) {
                            mbar_expect_tx(bar0 + 8 * e, G::TQ3_REC);
                            bulk_load(dst + e * G::SLOT, tq3_base + (size_t)list3[i] * hkv * G::TQ3_REC, G::TQ3_REC, bar0 + 8 * e);
                        } else mbar_arrive(bar0 + 8 * e);
                    }
                } else {
                    const int i = (ti - tiles3) * (kTile / 2) + wq;
                    if (i < n8) {
                        const uint8_t* rec = fp8_base + (size_t)(list8[i] & 0x7FFFFFF) * hkv * (2 * G::FP8_HALF);
                        mbar_expect_tx(bar0, G::FP8_HALF);
                        bulk_load(dst, rec, G::FP8_HALF, bar0);
                        mbar_expect_tx(bar0 + 8, G::FP8_HALF);
                        bulk_load(dst + G::SLOT, rec + G::FP8_HALF, G::FP8_HALF, bar0 + 8);
                    } else { mbar_arrive(bar0); mbar_arrive(bar0 + 8); }
                }
            };

            if (!worker) {
                // ================= issuing warp =================
                for (int ti = 0; ti < n_tiles; ++ti) {
                    const bool stale = ti < tiles3;
                    const int np = stale ? min(kTile, n3 - ti * kTile) : min(kTile / 2, n8 - (ti - tiles3) * (kTile / 2));
                    const uint32_t qtile = sbase + (stale ? G::OFF_QT : G::OFF_QF);
                    bar_sync(idK, 160);                      // first half of the key tile stored
                    tc_fence_after();
                    if (lane == 0) {
#pragma unroll 1
                        for (int kb = 0; kb < NB / 2; ++kb)
                            mma_ts(tb + kColS, tb + kColK + 8 * kb, b_tile_desc(qtile + kb * 512), kIdesc, kb > 0);
                    }
                    __syncwarp();
                    bar_sync(idK2, 160);                     // second half
                    tc_fence_after();
                    if (lane == 0) {
#pragma unroll 1
                        for (int kb = NB / 2; kb < NB; ++kb)
                            mma_ts(tb + kColS, tb + kColK + 8 * kb, b_tile_desc(qtile + kb * 512), kIdesc, 1);
                        mma_commit(bars + 8 * 16);
                    }
                    __syncwarp();
                    const int nb = (np + 1) / 2;
#pragma unroll 1
                    for (int bi = 0; bi < nb; ++bi) {
                        const uint32_t vb = bi & 1;
                        bar_sync(idV0 + vb, 160);            // value tiles of the batch stored (and, for the first, all P tiles)
                        tc_fence_after();
                        if (lane == 0) {
#pragma unroll 1
                            for (int e = 0; e < 2; ++e) {
                                const int p = 2 * bi + e;
                                if (p >= np) break;
                                const uint64_t dp = b_tile_desc(ptiles + p * 512);
#pragma unroll
                                for (int m = 0; m < 2; ++m)
                                    mma_ts(tb + kColT + vb * 64 + e * 32 + m * 16, tb + kColV + vb * 32 + e * 16 + m * 8, dp, kIdesc, 0);
                            }
                            mma_commit(bars + 8 * (17 + vb));
                        }
                        __syncwarp();
                    }
                }
            } else {
                // ================= worker warps =================
                if (n_tiles > 0) issue_tile(0, tcount & 1);
                for (int ti = 0; ti < n_tiles; ++ti) {
                    const bool stale = ti < tiles3;
                    const int first = stale ? ti * kTile : (ti - tiles3) * (kTile / 2);
                    const int np = stale ? min(kTile, n3 - first) : min(kTile / 2, n8 - first);
                    const uint32_t buf = tcount & 1, par = (tcount >> 1) & 1;
                    ++tcount;
                    const uint32_t tile = ring + buf * kTile * G::SLOT;
                    // every worker of the team has finished the tile before: the other buffer can be refilled now
                    bar_sync(idW, 128);
                    if (ti + 1 < n_tiles) issue_tile(ti + 1, tcount & 1);
#pragma unroll 1
                    for (int s = 0; s < kTile; ++s) wait_bar(bars + 8 * (buf * kTile + s), par);
                    failed = __any_sync(FULL, failed);
                    TM_STAMP(2);

                    // ---- keys of this warp's two pages -> tensor memory, in two halves of d ---------------------
#pragma unroll 1
                    for (int half = 0; half < 2; ++half) {
#pragma unroll 1
                        for (int e = 0; e < 2; ++e) {
                            const int p = 2 * wq + e;
                            if (p >= np) continue;
                            const uint32_t dst = tb + kColK + my_lanes + ((uint32_t)(16 * e) << 16) + 64 * half;
                            if (stale) {
                                // words 6 half .. 6 half + 5 of the lane: two 16-byte chunks (the second half starts mid-chunk)
                                const uint32_t sec = tile + p * G::SLOT + lane * 16;
                                const uint4 c0 = lds128(sec + (half ? 512 : 0)), c1 = lds128(sec + (half ? 1024 : 512));
                                const uint32_t kw[6] = {half ? c0.z : c0.x, half ? c0.w : c0.y, half ? c1.x : c0.z,
                                                        half ? c1.y : c0.w, half ? c1.z : c1.x, half ? c1.w : c1.y};
#pragma unroll
                                for (int j = 0; j < 2; ++j) {
                                    const uint32_t A = kw[3 * j], Bw = kw[3 * j + 1], Cw = kw[3 * j + 2];
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
#pragma unroll
                                for (int jj = 0; jj < 2; ++jj) {
                                    const int j = 2 * half + jj;
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
                                    tmem_st_frag4(dst + 32 * jj, r);
                                }
                            }
                        }
                        tmem_wait_st();
                        tc_fence_before();
                        bar_arrive(half ? idK2 : idK, 160);
                    }
                    TM_STAMP(3);

                    // ---- scores of this thread's token -------------------------------------------------------
                    const int p_me = 2 * wq + (lane >> 4), tok = lane & 15;
                    int valid = kPage;
                    if (!stale && p_me < np) { const int v = (list8[first + p_me] >> 27) & 15; valid = v ? v : kPage; }
                    const bool live = p_me < np && tok < valid;
                    wait_bar(bars + 8 * 16, scount & 1);
                    ++scount;
                    failed = __any_sync(FULL, failed);
                    TM_STAMP(4);
                    tc_fence_after();
                    float s[8];
                    {
                        float c[16];
                        tmem_ld16(tb + kColS + my_lanes, c);
                        tmem_wait_ld();
                        float rsc = sc2 * P.k_scale;
                        if (stale) {
                            const uint32_t gaddr = tile + (p_me < np ? p_me : 0) * G::SLOT + 12 * D;
                            rsc = __half2float(__ushort_as_half(lds16(gaddr + 2 * tok))) * sc2;
                        }
#pragma unroll
                        for (int i = 0; i < 8; ++i) s[i] = live ? (c[i] + c[8 + i]) * rsc : -CUDART_INF_F;
                    }
                    // running maxima: raised (for the whole team) only when some score exceeds them by 2^kRescaleSlack
                    bool ex = false;
#pragma unroll
                    for (int i = 0; i < 8; ++i) ex = ex || (s[i] > m_run[i] + kRescaleSlack);
                    ex = __any_sync(FULL, ex);
                    if (lane == 0) cnt[4 + wq] = ex ? 1 : 0;
                    bar_sync(idW, 128);
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
                        bar_sync(idW, 128);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float* q4 = reinterpret_cast<const float*>(cnt) + 8 + i;
                            const float nm = fmaxf(fmaxf(q4[0], q4[8]), fmaxf(q4[16], q4[24]));
                            if (nm > m_run[i] + kRescaleSlack) {
                                const float f = m_run[i] == -CUDART_INF_F ? 0.f : fast_exp2(m_run[i] - nm);
                                m_run[i] = nm;
                                l_run[i] *= f;
                                acc0[i] *= f;
                                acc1[i] *= f;
                            }
                        }
                        bar_sync(idW, 128);                  // the maxima are read before the next tile overwrites them
                    }
                    // probabilities of this token -> B tile of its page (rows 0-7 high, 8-15 low fp16 halves), page sums
                    {
                        const int kk = stale ? k_of_token_tq3(tok) : tok;
                        const uint32_t tp = ptiles + (p_me & (kTile - 1)) * 512;
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
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    }
                    bar_sync(idW, 128);                      // page sums and P tiles of all four warps are in place
                    TM_STAMP(5);

                    // ---- values: two pages at a time; the products of a batch run while the next one is unpacked -----
                    auto scale_batch = [&](int bi) {
                        const uint32_t vb = bi & 1;
                        TM_STAMP(6);
                        if (vb) { wait_bar(bars + 8 * 18, tcnt1 & 1); ++tcnt1; } else { wait_bar(bars + 8 * 17, tcnt0 & 1); ++tcnt0; }
                        TM_STAMP(7);
                        tc_fence_after();
#pragma unroll 1
                        for (int e = 0; e < 2; ++e) {
                            const int p = 2 * bi + e;
                            if (p >= np) break;
                            float t0[16], t1[16];
                            tmem_ld16(tb + kColT + vb * 64 + e * 32 + my_lanes, t0);
                            tmem_ld16(tb + kColT + vb * 64 + e * 32 + 16 + my_lanes, t1);
                            tmem_wait_ld();
                            const float4 pa = *reinterpret_cast<const float4*>(ps_s + p * 8), pb = *reinterpret_cast<const float4*>(ps_s + p * 8 + 4);
                            const float ps[8] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
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
                        TM_STAMP(8);
                    };
                    const int nb = (np + 1) / 2;
#pragma unroll 1
                    for (int bi = 0; bi < nb; ++bi) {
                        const uint32_t vb = bi & 1;
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
                        bar_arrive(idV0 + vb, 160);
                        if (bi > 0) scale_batch(bi - 1);
                    }
                    if (nb > 0) scale_batch(nb - 1);
                    failed = __any_sync(FULL, failed);
                }
            }
            bar_sync(idR, 160);                              // round finished: lists and counters may be rewritten
        }

        // ---- combine the teams of the block (ring memory is idle now) -------------------------------------
        TM_STAMP(9);
        tc_fence_before();
        __syncthreads();
        TM_STAMP(10);
        if (worker && ttid == 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i) sm_m[team * 8 + i] = m_run[i];
        }
        __syncthreads();
        if (worker) {
            const int c0 = 16 * (4 * wq + (lane >> 4)) + (lane & 15), c1 = c0 + 32;
            float f[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float M = -CUDART_INF_F;
#pragma unroll
                for (int u = 0; u < NU; ++u) M = fmaxf(M, sm_m[u * 8 + i]);
                f[i] = m_run[i] == -CUDART_INF_F ? 0.f : fast_exp2(m_run[i] - M);
            }
            float* mine = red + (size_t)team * D * 8;
            *reinterpret_cast<float4*>(mine + c0 * 8) = make_float4(acc0[0] * f[0], acc0[1] * f[1], acc0[2] * f[2], acc0[3] * f[3]);
            *reinterpret_cast<float4*>(mine + c0 * 8 + 4) = make_float4(acc0[4] * f[4], acc0[5] * f[5], acc0[6] * f[6], acc0[7] * f[7]);
            *reinterpret_cast<float4*>(mine + c1 * 8) = make_float4(acc1[0] * f[0], acc1[1] * f[1], acc1[2] * f[2], acc1[3] * f[3]);
            *reinterpret_cast<float4*>(mine + c1 * 8 + 4) = make_float4(acc1[4] * f[4], acc1[5] * f[5], acc1[6] * f[6], acc1[7] * f[7]);
            if (ttid == 0) {
#pragma unroll
                for (int i = 0; i < 8; ++i) sm_l[team * 8 + i] = l_run[i] * f[i];
            }
        }
        __syncthreads();

        const bool whole_row = (pos == row_start) && (pos + n_seg == row_end);
        if (whole_row) {
            for (int e = tid; e < 8 * D; e += NT) {
                const int head = e & 7, ch = e >> 3;
                if (head >= GQ) continue;
                float acc = 0.f, l = 0.f;
#pragma unroll
                for (int u = 0; u < NU; ++u) {
                    acc += red[(size_t)u * D * 8 + e];
                    l += sm_l[u * 8 + head];
                }
                P.out[((size_t)b * hq + h * GQ + head) * D + ch] = l > 0.f ? acc / l : 0.f;
            }
            if (P.lse && tid < GQ) {
                float l = 0.f, M = -CUDART_INF_F;
                for (int u = 0; u < NU; ++u) {
                    l += sm_l[u * 8 + tid];
                    M = fmaxf(M, sm_m[u * 8 + tid]);
                }
                P.lse[(size_t)b * hq + h * GQ + tid] = l > 0.f ? (M + log2f(l)) * kLn2 : -CUDART_INF_F;
            }
        } else {
            float* slot = P.partials + (size_t)(2 * blockIdx.x + (pos != my_start ? 1 : 0)) * (8 * D + 16);
            for (int e = tid; e < 8 * D; e += NT) {
                float acc = 0.f;
#pragma unroll
                for (int u = 0; u < NU; ++u) acc += red[(size_t)u * D * 8 + e];
                slot[e] = acc;
            }
            if (tid < 8) {
                float l = 0.f, M = -CUDART_INF_F;
                for (int u = 0; u < NU; ++u) {
                    l += sm_l[u * 8 + tid];
                    M = fmaxf(M, sm_m[u * 8 + tid]);
                }
                slot[8 * D + tid] = M;
                slot[8 * D + 8 + tid] = l;
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
                merge_row<D, NT>(P, first_slot, 2 * c0, n_parts, red, b, h);
            }
        }
        __syncthreads();
        TM_STAMP(11);
        pos += n_seg;
    }
#ifdef MKV_TIMELINE
    if (tid == 0) {
        for (int k = 0; k < 12; ++k) g_timeline[blockIdx.x * 16 + k] = tl_acc[k];
        g_timeline[blockIdx.x * 16 + 15] = tl_begin;
        g_timeline[blockIdx.x * 16 + 14] = tl_now();
    }
#endif
    tc_fence_before();
    __syncthreads();
    if (warp == kWorkerWarps) tmem_dealloc(tmem_all, 512);
}
#undef TM_STAMP
