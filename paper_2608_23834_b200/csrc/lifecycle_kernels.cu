// Append (bf16 -> e4m3 into Recent pages), Demote (FP8 page -> TQ3 record, then publish) and the
// Anchor tag flip.  Algorithm 1 steps 1-2; Section 4 "normalize-rotate-pack".
//
// The TQ3 encoder is specified as a sequence of single IEEE fp32 operations in a fixed order, so
// every arithmetic step below uses a round-to-nearest intrinsic (__fadd_rn, __fmul_rn, __fdiv_rn,
// __fsqrt_rn): the compiler may not fuse or reorder them.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include <cmath>

#include "mkv_internal.cuh"

namespace mkv {

__device__ __forceinline__ float e4m3_to_f32(uint8_t b)
{
    __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)b, __NV_E4M3);
    return __half2float(__half(h));
}

__device__ __forceinline__ uint16_t f32_to_f16_sat_bits(float x)
{
    x = fminf(fmaxf(x, -65504.f), 65504.f);
    return __half_as_ushort(__float2half_rn(x));
}

// ------------------------------------------------------------------------------------------ append
// One token of one KV head: thread i converts elements 2i, 2i+1 of K and V (scale, round to nearest
// even, saturate to +-448) and stores K token-major, V channel-major.
template <int D>
__device__ __forceinline__ void append_token(uint8_t* __restrict__ rec, int slot, float inv_k_scale, float inv_v_scale,
                                             const __nv_bfloat162* __restrict__ k, const __nv_bfloat162* __restrict__ v,
                                             int pair)
{
    float2 kf = __bfloat1622float2(k[pair]);
    float2 vf = __bfloat1622float2(v[pair]);
    kf.x = __fmul_rn(kf.x, inv_k_scale);
    kf.y = __fmul_rn(kf.y, inv_k_scale);
    vf.x = __fmul_rn(vf.x, inv_v_scale);
    vf.y = __fmul_rn(vf.y, inv_v_scale);
    const __nv_fp8x2_storage_t kq = __nv_cvt_float2_to_fp8x2(kf, __NV_SATFINITE, __NV_E4M3);
    const __nv_fp8x2_storage_t vq = __nv_cvt_float2_to_fp8x2(vf, __NV_SATFINITE, __NV_E4M3);
    const int i = 2 * pair;
    *reinterpret_cast<uint16_t*>(rec + slot * D + i) = kq;             // K: token-major
    rec[16 * D + i * kPage + slot] = (uint8_t)(vq & 0xFF);             // V: channel-major
    rec[16 * D + (i + 1) * kPage + slot] = (uint8_t)(vq >> 8);
}

// Decode-sized calls: one block per (token, KV head).
template <int D>
__global__ void __launch_bounds__(D / 2) append_kernel(uint8_t* __restrict__ fp8, int fp8_pages, int hkv, int tiles,
                                                        float inv_k_scale, float inv_v_scale,
                                                        const __nv_bfloat162* __restrict__ k,
                                                        const __nv_bfloat162* __restrict__ v,
                                                        const int32_t* __restrict__ slots,
                                                        uint32_t* __restrict__ status)
{
    const int tok = blockIdx.x, h = blockIdx.y;
    const int sm = slots[tok];
    if (sm < 0) return;
    // slot_mapping = page * page_tokens + position; a page is `tiles` consecutive 16-token records per head
    const int gt = sm >> 4, slot = sm & 15, page = gt / tiles, m = gt - page * tiles;
    if (page >= fp8_pages) {
        if (threadIdx.x == 0) atomicOr(status, kStBounds);
        return;
    }
    uint8_t* rec = fp8 + (((size_t)page * hkv + h) * tiles + m) * fp8_record_bytes(D);
    const size_t src = ((size_t)tok * hkv + h) * (D / 2);
    append_token<D>(rec, slot, inv_k_scale, inv_v_scale, k + src, v + src, threadIdx.x);
}

// eight bf16 (one 16-byte load) -> eight e4m3 bytes
__device__ __forceinline__ uint2 bf16x8_to_e4m3x8(uint4 in, float inv_scale)
{
    const uint32_t w[4] = {in.x, in.y, in.z, in.w};
    uint32_t q[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
        f.x = __fmul_rn(f.x, inv_scale);
        f.y = __fmul_rn(f.y, inv_scale);
        q[i] = __nv_cvt_float2_to_fp8x2(f, __NV_SATFINITE, __NV_E4M3);
    }
    return make_uint2(q[0] | (q[1] << 16), q[2] | (q[3] << 16));
}

// Prefill-sized calls: one block per (16 consecutive input tokens, KV head).  Where the 16 tokens fill
// one page front to back (slot_mapping[t0 + i] = 16 page + i), K rows leave with 8-byte stores and V
// is transposed through shared memory so that every channel's 16 tokens leave as one 16-byte store;
// any other group (skipped tokens, a run that starts inside a page, the tail) takes the per-token path.
template <int D>
__global__ void __launch_bounds__(128) append_run_kernel(uint8_t* __restrict__ fp8, int fp8_pages, int hkv, int tiles,
                                                          float inv_k_scale, float inv_v_scale,
                                                          const __nv_bfloat162* __restrict__ k,
                                                          const __nv_bfloat162* __restrict__ v,
                                                          const int32_t* __restrict__ slots, int n,
                                                          uint32_t* __restrict__ status)
{
    constexpr int VROW = D + 4;                      // padded token row of the transposition tile
    __shared__ __align__(16) uint8_t vt[kPage * VROW];
    __shared__ int32_t slot_s[kPage];
    __shared__ int run_s;
    const int t0 = blockIdx.x * kPage, h = blockIdx.y, tid = threadIdx.x;
    const int cnt = min(kPage, n - t0);
    if (tid < kPage) slot_s[tid] = tid < cnt ? slots[t0 + tid] : -1;
    __syncthreads();
    if (tid == 0) {
        const int s0 = slot_s[0];
        bool run = cnt == kPage && s0 >= 0 && (s0 & 15) == 0 && (s0 >> 4) / tiles < fp8_pages;
        for (int i = 1; run && i < kPage; ++i) run = slot_s[i] == s0 + i;
        run_s = run ? 1 : 0;
    }
    __syncthreads();
    if (run_s) {
        const int gt = slot_s[0] >> 4, page = gt / tiles;
        uint8_t* rec = fp8 + (((size_t)page * hkv + h) * tiles + (gt - page * tiles)) * fp8_record_bytes(D);
        constexpr int CPT = D / 8;                   // 16-byte input chunks per token
        for (int c = tid; c < kPage * CPT; c += 128) {
            const int t = c / CPT, c8 = c % CPT;
            const size_t at = ((size_t)(t0 + t) * hkv + h) * (D / 8) + c8;
            const uint2 kq = bf16x8_to_e4m3x8(reinterpret_cast<const uint4*>(k)[at], inv_k_scale);
            const uint2 vq = bf16x8_to_e4m3x8(reinterpret_cast<const uint4*>(v)[at], inv_v_scale);
            *reinterpret_cast<uint2*>(rec + t * D + 8 * c8) = kq;
            *reinterpret_cast<uint32_t*>(vt + t * VROW + 8 * c8) = vq.x;
            *reinterpret_cast<uint32_t*>(vt + t * VROW + 8 * c8 + 4) = vq.y;
        }
        __syncthreads();
        // thread c4 owns channels 4 c4 .. 4 c4 + 3: 16 words (one per token) -> 4 x 16 bytes
        for (int c4 = tid; c4 < D / 4; c4 += 128) {
            uint32_t w[kPage];
#pragma unroll
            for (int t = 0; t < kPage; ++t) w[t] = *reinterpret_cast<const uint32_t*>(vt + t * VROW + 4 * c4);
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                uint32_t o[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint32_t lo = __byte_perm(w[4 * q], w[4 * q + 1], 0x0040 + 0x0011 * ch);   // bytes ch of t, t+1
                    const uint32_t hi = __byte_perm(w[4 * q + 2], w[4 * q + 3], 0x0040 + 0x0011 * ch);
                    o[q] = __byte_perm(lo, hi, 0x5410);
                }
                *reinterpret_cast<uint4*>(rec + 16 * D + (4 * c4 + ch) * kPage) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
        return;
    }
    for (int t = 0; t < cnt; ++t) {
        const int sm = slot_s[t];
        if (sm < 0) continue;
        const int gt = sm >> 4, page = gt / tiles;
        if (page >= fp8_pages) {
            if (tid == 0) atomicOr(status, kStBounds);
            continue;
        }
        uint8_t* rec = fp8 + (((size_t)page * hkv + h) * tiles + (gt - page * tiles)) * fp8_record_bytes(D);
        const size_t src = ((size_t)(t0 + t) * hkv + h) * (D / 2);
        if (tid < D / 2) append_token<D>(rec, sm & 15, inv_k_scale, inv_v_scale, k + src, v + src, tid);
    }
}

// Decode-sized append into the pools of several layers: one block per (token, KV head, layer).
struct AppendLayers {
    uint8_t* fp8[MKV_MAX_LAYERS_PER_CALL];
    const __nv_bfloat162* k[MKV_MAX_LAYERS_PER_CALL];
    const __nv_bfloat162* v[MKV_MAX_LAYERS_PER_CALL];
    uint32_t* status[MKV_MAX_LAYERS_PER_CALL];
    float inv_k_scale[MKV_MAX_LAYERS_PER_CALL], inv_v_scale[MKV_MAX_LAYERS_PER_CALL];
    int fp8_pages[MKV_MAX_LAYERS_PER_CALL];
};

template <int D>
__global__ void __launch_bounds__(D / 2) append_layers_kernel(const AppendLayers A, int hkv, int tiles,
                                                               const int32_t* __restrict__ slots)
{
    const int tok = blockIdx.x, h = blockIdx.y, layer = blockIdx.z;
    const int sm = slots[tok];
    if (sm < 0) return;
    const int gt = sm >> 4, slot = sm & 15, page = gt / tiles, m = gt - page * tiles;
    if (page >= A.fp8_pages[layer]) {
        if (threadIdx.x == 0) atomicOr(A.status[layer], kStBounds);
        return;
    }
    uint8_t* rec = A.fp8[layer] + (((size_t)page * hkv + h) * tiles + m) * fp8_record_bytes(D);
    const size_t src = ((size_t)tok * hkv + h) * (D / 2);
    append_token<D>(rec, slot, A.inv_k_scale[layer], A.inv_v_scale[layer], A.k[layer] + src, A.v[layer] + src, threadIdx.x);
}

int32_t launch_append_layers(mkv_pool* const* pools, const void* const* k, const void* const* v, const int32_t* slots,
                             int n, int n_layers, cudaStream_t s)
{
    AppendLayers A;
    for (int i = 0; i < n_layers; ++i) {
        A.fp8[i] = pools[i]->fp8;
        A.k[i] = static_cast<const __nv_bfloat162*>(k[i]);
        A.v[i] = static_cast<const __nv_bfloat162*>(v[i]);
        A.status[i] = pools[i]->status_dev;
        A.inv_k_scale[i] = 1.0f / pools[i]->cfg.k_scale;
        A.inv_v_scale[i] = 1.0f / pools[i]->cfg.v_scale;
        A.fp8_pages[i] = pools[i]->cfg.fp8_pages;
    }
    const mkv_pool* p = pools[0];
    dim3 grid(n, p->hkv, n_layers);
    if (p->d == 128) append_layers_kernel<128><<<grid, 64, 0, s>>>(A, p->hkv, p->tiles, slots);
    else append_layers_kernel<256><<<grid, 128, 0, s>>>(A, p->hkv, p->tiles, slots);
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
}

int32_t launch_append(mkv_pool* p, const void* k, const void* v, const int32_t* slots, int n, cudaStream_t s)
{
    const float ik = 1.0f / p->cfg.k_scale, iv = 1.0f / p->cfg.v_scale;
    const __nv_bfloat162* kk = (const __nv_bfloat162*)k;
    const __nv_bfloat162* vv = (const __nv_bfloat162*)v;
    if (n >= 2 * kPage) {
        dim3 grid((n + kPage - 1) / kPage, p->hkv);
        if (p->d == 128)
            append_run_kernel<128><<<grid, 128, 0, s>>>(p->fp8, p->cfg.fp8_pages, p->hkv, p->tiles, ik, iv, kk, vv, slots, n,
                                                        p->status_dev);
        else
            append_run_kernel<256><<<grid, 128, 0, s>>>(p->fp8, p->cfg.fp8_pages, p->hkv, p->tiles, ik, iv, kk, vv, slots, n,
                                                        p->status_dev);
    } else {
        dim3 grid(n, p->hkv);
        if (p->d == 128)
            append_kernel<128><<<grid, 64, 0, s>>>(p->fp8, p->cfg.fp8_pages, p->hkv, p->tiles, ik, iv, kk, vv, slots, p->status_dev);
        else
            append_kernel<256><<<grid, 128, 0, s>>>(p->fp8, p->cfg.fp8_pages, p->hkv, p->tiles, ik, iv, kk, vv, slots, p->status_dev);
    }
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
}

// ---- thread-block cluster helpers (Demote and Promote run one cluster per page) ------------------
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_size()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
// Every thread of every block of the cluster arrives exactly once; no block leaves early.
__device__ __forceinline__ void cluster_barrier()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Blocks per page.  A call of few pages (the retier of a decode step) is latency-bound: the heads of a
// page go to the blocks of a cluster, the largest divisor of the head count that a portable cluster
// allows.  A call that fills the GPU with one block per page anyway keeps the heads in one block, which
// amortises the per-block set-up and overlaps one head's copy-out with the next head's encoding.
static int heads_cluster(int hkv, int n_pages)
{
    if (n_pages > 2 * 148) return 1;
    for (int c = 8; c > 1; --c)
        if (hkv % c == 0) return c;
    return 1;
}

template <typename Kernel, typename... Args>
static cudaError_t launch_clustered(Kernel kernel, int n_pages, int csize, int threads, cudaStream_t s, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_pages * csize);
    cfg.blockDim = dim3(threads);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = csize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// ------------------------------------------------------------------------------------------ demote
// One thread-block cluster per page, its blocks sharing out the KV heads (block r takes heads r,
// r + cluster size, ...); the cluster's barrier orders every head's record before the page is
// published.  Warps encode key vectors (one token each), threads encode value channels; the 3-bit
// codes meet in shared memory, where every thread assembles one word triple of the record image; the
// image leaves with 16-byte stores.
//
// Shared layout: key codes [token][D + 8] (the 8 pad bytes spread the token rows over the banks for
// the packers, which read rows g and g + 8), value codes [channel][16 tokens], and two record images
// (alternating per head, so that the copy-out of one head overlaps the encoding of the next).

// 16 bytes global -> shared, asynchronously (both addresses 16-byte aligned); completion by cp.async.wait_all
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
                 : "memory");
}

// Two fp32 values in one 64-bit register and the packed operations on them (add, mul, fma, each half rounded to
// nearest even exactly like the scalar instruction): half the instructions for element-wise arithmetic.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b)
{
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b)
{
    f32x2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c)
{
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

// two e4m3 bytes (low byte first) -> two fp32
__device__ __forceinline__ float2 e4m3x2_to_f32(uint32_t two_bytes)
{
    const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)two_bytes, __NV_E4M3);
    return __half22float2(__half2(h));
}

// nibble pairs of two bytes -> one byte: (x & 0x000F) | ((x & 0x0F00) >> 4)
__device__ __forceinline__ uint32_t squeeze_nibbles(uint32_t x) { return (x & 0xFu) | ((x >> 4) & 0xF0u); }

// four code bytes -> four nibbles
__device__ __forceinline__ uint32_t squeeze4(uint32_t x)
{
    return (x & 0xFu) | ((x >> 4) & 0xF0u) | ((x >> 8) & 0xF00u) | ((x >> 12) & 0xF000u);
}

// Pages of several tiles are converted by gridDim.y clusters per page (rows of tiles).  When the call publishes
// from inside the kernel, every cluster draws a ticket of its page once all its tiles are written and fenced
// (called by thread 0 of the cluster's first block after the cluster barrier); the cluster that draws the last
// one publishes and leaves the counter at zero.  Nobody waits.  Without tickets (16-token pages: one cluster
// per page) every caller is the last.
__device__ __forceinline__ bool last_cluster_of_page(uint32_t* page_tickets, int page)
{
    if (page_tickets == nullptr) return true;
    const uint32_t prev = atomicAdd(page_tickets + page, 1u);
    if (prev != gridDim.y - 1) return false;
    __threadfence();                    // the other clusters' tiles are ordered before what this thread writes next
    page_tickets[page] = 0u;
    return true;
}

// Constants of the key encoder that depend only on the lane (FMT: the record format's codebook).
template <int D, int FMT>
struct DemoteLane {
    float c0sq, c1sq, c2sq, c3sq;     // squared levels (single fp32 products, as the record's norm correction defines them)
    uint32_t flip[D / 32];            // rotation signs of this lane's key elements, as fp32 sign-bit masks
    float sgn[5];                     // butterfly stage m: lanes with bit m set subtract (-1.0f), the others add (+1.0f)
    __device__ __forceinline__ void init(const SigmaBits& sigma, int lane)
    {
        using CB = KeyCodebook<FMT>;
        c0sq = __fmul_rn(CB::C0, CB::C0);
        c1sq = __fmul_rn(CB::C1, CB::C1);
        c2sq = __fmul_rn(CB::C2, CB::C2);
        c3sq = __fmul_rn(CB::C3, CB::C3);
#pragma unroll
        for (int r = 0; r < D / 32; ++r) {
            const int i = lane * (D / 32) + r;
            flip[r] = ((sigma.w[i >> 5] >> (i & 31)) & 1u) << 31;
        }
#pragma unroll
        for (int b = 0; b < 5; ++b) sgn[b] = ((lane >> b) & 1) ? -1.0f : 1.0f;
    }
};

// Encodes the 16 tokens of one FP8 record (rec8) into the record image img = [key codes | value codes | g |
// scale/zero] in shared memory; all D threads of the block call it.  OWN_META: the value scale and zero come
// from these 16 tokens (16-token pages); otherwise thread c passes the page's scale/zero of channel c.
template <int D, bool OWN_META, int FMT>
__device__ __forceinline__ void demote_tile(const uint8_t* __restrict__ rec8, uint8_t* img, uint8_t* kcode, uint8_t* vcode,
                                            const DemoteLane<D, FMT>& K, float k_scale, float v_scale, uint16_t sc_page,
                                            uint16_t zp_page)
{
    using CB = KeyCodebook<FMT>;
    constexpr int EPL = D / 32, NJ = D / 64, KROW = D + 8, NT = D;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const float c0sq = K.c0sq, c1sq = K.c1sq, c2sq = K.c2sq, c3sq = K.c3sq;
    const uint32_t (&flip)[EPL] = K.flip;
    const float (&sgn)[5] = K.sgn;
    // ---- keys: warp w encodes tokens w, w + NT/32, ... ------------------------------------------
    for (int tok = warp; tok < kPage; tok += NT / 32) {
        float x[EPL], a[EPL];
        uint32_t raw[EPL / 4];
        if constexpr (EPL == 8) {
            const uint2 u = *reinterpret_cast<const uint2*>(rec8 + tok * D + lane * EPL);
            raw[0] = u.x;
            raw[1] = u.y;
        } else {
            raw[0] = *reinterpret_cast<const uint32_t*>(rec8 + tok * D + lane * EPL);
        }
#pragma unroll
        for (int r = 0; r < EPL; r += 2) {
            const float2 f = e4m3x2_to_f32((raw[r >> 2] >> (8 * (r & 3))) & 0xFFFFu);
            x[r] = f.x;
            x[r + 1] = f.y;
        }
        if (k_scale != 1.0f) {           // a product with 1 is the factor itself: the common case skips it
#pragma unroll
            for (int r = 0; r < EPL; ++r) x[r] = __fmul_rn(x[r], k_scale);
        }
#pragma unroll
        for (int r = 0; r < EPL; ++r) a[r] = __uint_as_float(__float_as_uint(x[r]) ^ flip[r]);
        // Walsh-Hadamard butterflies, strides ascending: inside the lane, then across lanes
        // (stride 1 pairs neighbours: scalar; from stride 2 on two butterflies share one packed instruction)
#pragma unroll
        for (int r = 0; r < EPL; r += 2) {
            const float u = a[r], w = a[r + 1];
            a[r] = __fadd_rn(u, w);
            a[r + 1] = __fsub_rn(u, w);
        }
        f32x2 ap[EPL / 2];
        const f32x2 minus1 = pack2(-1.0f, -1.0f);
#pragma unroll
        for (int r = 0; r < EPL / 2; ++r) ap[r] = pack2(a[2 * r], a[2 * r + 1]);
#pragma unroll
        for (int hh = 1; hh < EPL / 2; hh <<= 1)            // strides 2, 4 of the elements = 1, 2 of the pairs
#pragma unroll
            for (int r = 0; r < EPL / 2; ++r)
                if ((r & hh) == 0) {
                    const f32x2 u = ap[r], w = ap[r + hh];
                    ap[r] = add2(u, w);
                    ap[r + hh] = fma2(w, minus1, u);        // u - w: the product with -1 is exact, one rounding
                }
#pragma unroll
        for (int b = 0; b < 5; ++b) {
            const f32x2 s2 = pack2(sgn[b], sgn[b]);
#pragma unroll
            for (int r = 0; r < EPL / 2; ++r) {
                // lower lane: o + a; upper lane: o - a.  The product with +-1 is exact, so the fused form rounds
                // once, exactly like the single addition it stands for (zero signs included)
                float lo, hi;
                unpack2(ap[r], lo, hi);
                const float olo = __shfl_xor_sync(0xffffffffu, lo, 1 << b), ohi = __shfl_xor_sync(0xffffffffu, hi, 1 << b);
                ap[r] = fma2(ap[r], s2, pack2(olo, ohi));
            }
        }
#pragma unroll
        for (int r = 0; r < EPL / 2; ++r) unpack2(ap[r], a[2 * r], a[2 * r + 1]);
        // |x|^2: pairwise tree in index order (every element of the butterfly ends equal)
        float e[EPL];
#pragma unroll
        for (int r = 0; r < EPL; r += 2) {
            const f32x2 xx = pack2(x[r], x[r + 1]);
            unpack2(mul2(xx, xx), e[r], e[r + 1]);
        }
#pragma unroll
        for (int hh = 1; hh < EPL; hh <<= 1)
#pragma unroll
            for (int r = 0; r < EPL; r += 2 * hh) e[r] = __fadd_rn(e[r], e[r + hh]);
        float n2 = e[0];
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) n2 = __fadd_rn(n2, __shfl_xor_sync(0xffffffffu, n2, m));
        const float nx = __fsqrt_rn(n2);
        const float t1 = __fmul_rn(CB::B0, nx), t2 = __fmul_rn(CB::B1, nx), t3 = __fmul_rn(CB::B2, nx);
        float f[EPL];
        uint32_t packed[EPL / 4];
        uint32_t sq64 = 4u * EPL;          // record format 2: 64 x the sum of this lane's squared levels (4, 36, 121, 324)
#pragma unroll
        for (int r = 0; r < EPL / 4; ++r) packed[r] = 0;
#pragma unroll
        for (int r = 0; r < EPL; ++r) {
            const float w = fabsf(a[r]);
            const bool g1 = w > t1, g2 = w > t2, g3 = w > t3;
            // sign bit of the code: a[r] < 0 (a zero of either sign is positive)
            uint32_t code = a[r] < 0.0f ? 4u : 0u;
            if (g1) code += 1u;
            if (g2) code += 1u;
            if (g3) code += 1u;
            packed[r >> 2] |= code << (8 * (r & 3));
            if constexpr (FMT == 2) {
                if (g1) sq64 += 32u;
                if (g2) sq64 += 85u;
                if (g3) sq64 += 203u;
            } else {
                f[r] = g2 ? (g3 ? c3sq : c2sq) : (g1 ? c1sq : c0sq);
            }
        }
        if constexpr (EPL == 8)
            *reinterpret_cast<uint2*>(kcode + tok * KROW + lane * EPL) = make_uint2(packed[0], packed[1]);
        else
            *reinterpret_cast<uint32_t*>(kcode + tok * KROW + lane * EPL) = packed[0];
        float nc2;
        if constexpr (FMT == 2) {
            // The squared levels of format 2 are multiples of 1/64 and d of them sum to at most 5.0625 d, so every
            // partial sum of the pairwise tree is exact in fp32: any order gives the same bits, and the sum can be
            // taken in integers (one warp reduction) instead.
            static_assert(324 * D < (1 << 24), "exact in fp32");
            nc2 = __fmul_rn((float)__reduce_add_sync(0xffffffffu, sq64), 0.015625f);
        } else {
#pragma unroll
            for (int hh = 1; hh < EPL; hh <<= 1)
#pragma unroll
                for (int r = 0; r < EPL; r += 2 * hh) f[r] = __fadd_rn(f[r], f[r + hh]);
            nc2 = f[0];
#pragma unroll
            for (int m = 1; m < 32; m <<= 1) nc2 = __fadd_rn(nc2, __shfl_xor_sync(0xffffffffu, nc2, m));
        }
        const float nc = __fsqrt_rn(nc2);
        if (lane == 0)
            *reinterpret_cast<uint16_t*>(img + 12 * D + 2 * tok) =
                (nx == 0.0f) ? (uint16_t)0 : f32_to_f16_sat_bits(__fdiv_rn(nx, nc));
    }

    // ---- values: one thread per channel, 16 tokens of the page ------------------------------
    for (int c = tid; c < D; c += NT) {
        const uint4 raw = *reinterpret_cast<const uint4*>(rec8 + 16 * D + c * kPage);
        const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
        float val[kPage];
#pragma unroll
        for (int t = 0; t < kPage; t += 2) {
            const float2 f = e4m3x2_to_f32((rw[t >> 2] >> (8 * (t & 3))) & 0xFFFFu);
            val[t] = f.x;
            val[t + 1] = f.y;
        }
        if (v_scale != 1.0f) {
#pragma unroll
            for (int t = 0; t < kPage; ++t) val[t] = __fmul_rn(val[t], v_scale);
        }
        // scale and zero of the channel: from this tile's 16 tokens (16-token pages), or the page's (given)
        uint16_t sc = sc_page, zp = zp_page;
        if constexpr (OWN_META) {
            // minimum and maximum by strict comparison in token order.  The min/max instructions give the same
            // value except for the sign of a zero extreme and a leading NaN; those cases take the literal loop
            float mn = val[0], mx = val[0];
#pragma unroll
            for (int t = 1; t < kPage; ++t) {
                mn = fminf(mn, val[t]);
                mx = fmaxf(mx, val[t]);
            }
            if (!(mn != 0.0f && mx != 0.0f) || val[0] != val[0]) {
                mn = val[0];
                mx = val[0];
#pragma unroll
                for (int t = 1; t < kPage; ++t) {
                    if (val[t] < mn) mn = val[t];
                    if (val[t] > mx) mx = val[t];
                }
            }
            sc = f32_to_f16_sat_bits(__fdiv_rn(__fsub_rn(mx, mn), 7.0f));
            zp = f32_to_f16_sat_bits(mn);
        }
        const float scf = __half2float(__ushort_as_half(sc)), zpf = __half2float(__ushort_as_half(zp));
        {
            const int cb = c >> 4, row = c & 15;
            uint16_t* meta = reinterpret_cast<uint16_t*>(img + 12 * D + 32);
            const int hi = (cb >> 1) * 64 + (row & 7) * 8 + 4 * (cb & 1) + (row >> 3);
            meta[hi] = sc;
            meta[hi + 2] = zp;
        }
        // q = clamp(rint((val - zp) / sc), 0, 7), 0 when sc == 0, the division correctly rounded.
        // The correctly rounded quotient d = RN(num / sc) without the divider: with y = RN(1 / sc) (one correctly
        // rounded reciprocal per channel), q0 = RN(num y) is within 1.5 ulp of the quotient, one residual step
        // q1 = RN(q0 + (num - sc q0) y) makes it faithful, and for a faithful q1 the second step gives exactly d
        // (Markstein's theorem; the residuals are exact in an FMA).  No intermediate can overflow or underflow when
        // the value scale is between 2^-20 and 2^20 (numerators are 0 or at least 2^-52 and below 2^30, scales are
        // fp16 numbers); other scales take the divider.  A zero scale gives y = 0 and code 0, a zero numerator code 0,
        // a NaN input code 0, all as the quotient form does.
        const float den = scf != 0.0f ? scf : 1.0f;
        uint32_t q4[4] = {0u, 0u, 0u, 0u};
        if (v_scale >= 9.5367431640625e-07f && v_scale <= 1048576.0f) {
            const float y = scf != 0.0f ? __frcp_rn(scf) : 0.0f;
            // two tokens per instruction: the packed fp32 operations round each half like the scalar ones
            const f32x2 y2 = pack2(y, y), nden2 = pack2(-den, -den), nzp2 = pack2(-zpf, -zpf);
#pragma unroll
            for (int t = 0; t < kPage; t += 2) {
                const f32x2 num = add2(pack2(val[t], val[t + 1]), nzp2);           // val - zp (= val + (-zp), one rounding)
                const f32x2 q0 = mul2(num, y2);
                const f32x2 q1 = fma2(fma2(nden2, q0, num), y2, q0);
                const f32x2 d2 = fma2(fma2(nden2, q1, num), y2, q1);
                float d0, d1;
                unpack2(d2, d0, d1);
                const float r0 = fminf(fmaxf(rintf(d0), 0.0f), 7.0f);        // half to even; NaN -> 0
                const float r1 = fminf(fmaxf(rintf(d1), 0.0f), 7.0f);
                q4[t >> 2] |= ((uint32_t)(int)r0 << (8 * (t & 3))) | ((uint32_t)(int)r1 << (8 * ((t + 1) & 3)));
            }
        } else {
#pragma unroll
            for (int t = 0; t < kPage; ++t) {
                const float num = __fsub_rn(val[t], zpf);
                float r = rintf(__fdiv_rn(num != 0.0f ? num : den, den));   // half to even
                r = r < 0.0f ? 0.0f : r;
                r = r > 7.0f ? 7.0f : r;
                const uint32_t q = (num != 0.0f && scf != 0.0f) ? (uint32_t)(int)r : 0u;
                q4[t >> 2] |= q << (8 * (t & 3));
            }
        }
        *reinterpret_cast<uint4*>(vcode + c * kPage) = make_uint4(q4[0], q4[1], q4[2], q4[3]);
    }
    __syncthreads();

    // ---- pack: one thread per (section, triple j, fragment lane L) --------------------------
    for (int item = tid; item < 2 * NJ * 32; item += NT) {
        const int L = item & 31, j = (item >> 5) % NJ, section = item / (32 * NJ);
        const int g = L >> 2, tq = L & 3;
        uint32_t w0 = 0, w1 = 0, w2 = 0;
        if (section == 0 && FMT == 2) {
            // record format 2: register e = 4 (step % 2) + 2 u + b of the triple holds, in its four nibbles, the
            // codes of token g + 8u at dims 32 step + 16 b + 4 tq .. + 3 (steps 2j, 2j+1).  A: registers 0,1 with
            // the signs of 4,5; B: registers 2,3 with the signs of 6,7; C: magnitudes of 4,5 (low pair), 6,7 (high).
            uint32_t x[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
                x[e] = *reinterpret_cast<const uint32_t*>(kcode + (g + 8 * ((e >> 1) & 1)) * KROW + 32 * (2 * j + (e >> 2)) +
                                                          16 * (e & 1) + 4 * tq);
            auto signs = [](uint32_t v) { return squeeze4((v >> 2) & 0x01010101u) << 3; };
            auto mags = [](uint32_t v) { return squeeze4(v & 0x03030303u); };
            w0 = squeeze4(x[0]) | (squeeze4(x[1]) << 16) | signs(x[4]) | (signs(x[5]) << 16);
            w1 = squeeze4(x[2]) | (squeeze4(x[3]) << 16) | signs(x[6]) | (signs(x[7]) << 16);
            w2 = mags(x[4]) | (mags(x[5]) << 16) | ((mags(x[6]) | (mags(x[7]) << 16)) << 2);
        } else if (section == 0) {
            // key codes: nibble n = 2r + half holds row g + 8(r&1), slot 2tq + 8(r>>1) + half.
            // A: block 4j with the signs of block 4j+2; B: block 4j+1 with the signs of 4j+3;
            // C: magnitudes of blocks 4j+2 (low pair) and 4j+3 (high pair).
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const uint8_t* at = kcode + (g + 8 * (r & 1)) * KROW + 64 * j + 2 * tq + 8 * (r >> 1);
                const uint32_t b0 = *reinterpret_cast<const uint16_t*>(at);        // (half 0, half 1)
                const uint32_t b1 = *reinterpret_cast<const uint16_t*>(at + 16);
                const uint32_t b2 = *reinterpret_cast<const uint16_t*>(at + 32);
                const uint32_t b3 = *reinterpret_cast<const uint16_t*>(at + 48);
                w0 |= squeeze_nibbles(b0 | ((b2 & 0x0404u) << 1)) << (8 * r);
                w1 |= squeeze_nibbles(b1 | ((b3 & 0x0404u) << 1)) << (8 * r);
                w2 |= squeeze_nibbles((b2 & 0x0303u) | ((b3 & 0x0303u) << 2)) << (8 * r);
            }
        } else {
            // value codes: four 24-bit streams (group, half) per triple; stream code k is
            // channel block 4j + 2 grp + (k>>2), row g + 8(k&1), token 2tq + 8((k>>1)&1) + half
            uint32_t S[2][2] = {{0u, 0u}, {0u, 0u}};
#pragma unroll
            for (int grp = 0; grp < 2; ++grp)
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int cb = 4 * j + 2 * grp + (k >> 2), r = k & 3;
                    const uint32_t two = *reinterpret_cast<const uint16_t*>(
                        vcode + (16 * cb + g + 8 * (r & 1)) * kPage + 2 * tq + 8 * (r >> 1));
                    S[grp][0] |= (two & 7u) << (3 * k);
                    S[grp][1] |= (two >> 8) << (3 * k);
                }
            w0 = (S[0][0] & 0xFFFFu) | (S[0][1] << 16);
            w1 = (S[0][0] >> 16) | ((S[1][0] & 0xFFu) << 8) | ((S[0][1] >> 16) << 16) | (S[1][1] << 24);
            w2 = (S[1][0] >> 8) | ((S[1][1] >> 8) << 16);
        }
        uint8_t* sec = img + section * 6 * D;
        *reinterpret_cast<uint32_t*>(sec + lane_word_offset(D, L, 3 * j)) = w0;
        *reinterpret_cast<uint32_t*>(sec + lane_word_offset(D, L, 3 * j + 1)) = w1;
        *reinterpret_cast<uint32_t*>(sec + lane_word_offset(D, L, 3 * j + 2)) = w2;
    }
    __syncthreads();
}

template <int D, bool BIG, int FMT>
__global__ void __launch_bounds__(D) demote_kernel(const uint8_t* __restrict__ fp8, uint8_t* __restrict__ tq3,
                                                      int fp8_pages, int tq3_pages, int hkv, int tiles, float k_scale,
                                                      float v_scale, SigmaBits sigma,
                                                      const int32_t* __restrict__ src_ids,
                                                      const int32_t* __restrict__ dst_ids, int32_t* block_table,
                                                      uint8_t* tier_tag, const int64_t* entry_index, int64_t n_entries,
                                                      uint32_t* __restrict__ status, uint32_t* page_tickets)
{
    constexpr int KROW = D + 8;          // padded row of the key-code tile
    constexpr int REC = 16 * D + 32;     // bytes of one TQ3 record
    constexpr int NT = D;                // threads: one per value channel, one per packed word triple
    __shared__ __align__(16) uint8_t kcode[kPage * KROW];
    __shared__ __align__(16) uint8_t vcode[D * kPage];
    __shared__ __align__(16) uint8_t image[2][REC];

    const int csize = (int)cluster_size(), crank = (int)cluster_rank();
    const int page = blockIdx.x / csize, tid = threadIdx.x, lane = tid & 31;
    const int src = src_ids[page], dst = dst_ids[page];
    const bool valid = src >= 0 && src < fp8_pages && dst >= 0 && dst < tq3_pages;
    if (!valid && tid == 0 && crank == 0 && blockIdx.y == 0) atomicOr(status, kStBounds);
    DemoteLane<D, FMT> lane_consts;
    lane_consts.init(sigma, lane);

    int it = 0;
    for (int h = crank; valid && h < hkv; h += csize) {
        if constexpr (!BIG) {
            const uint8_t* rec8 = fp8 + ((size_t)src * hkv + h) * fp8_record_bytes(D);
            uint8_t* rec3 = tq3 + ((size_t)dst * hkv + h) * tq3_record_bytes(D);
            uint8_t* img = image[it++ & 1];
            demote_tile<D, true, FMT>(rec8, img, kcode, vcode, lane_consts, k_scale, v_scale, 0, 0);
            for (int i = tid; i < REC / 16; i += NT)
                reinterpret_cast<uint4*>(rec3)[i] = reinterpret_cast<const uint4*>(img)[i];
        } else {
            // pages of several tiles: the page's scale/zero were written by demote_minmax_kernel; the blocks of
            // grid row y take tiles y, y + gridDim.y, ... and write the tile part of the image only
            constexpr int TILE = 12 * D + 32;
            uint8_t* page3 = tq3 + ((size_t)dst * hkv + h) * tq3_page_bytes(D, tiles);
            const uint16_t* meta = reinterpret_cast<const uint16_t*>(page3 + (size_t)tiles * TILE);
            const int cb = tid >> 4, row = tid & 15;
            const int hi = (cb >> 1) * 64 + (row & 7) * 8 + 4 * (cb & 1) + (row >> 3);
            const uint16_t sc = meta[hi], zp = meta[hi + 2];
            for (int m = blockIdx.y; m < tiles; m += gridDim.y) {
                const uint8_t* rec8 = fp8 + (((size_t)src * hkv + h) * tiles + m) * fp8_record_bytes(D);
                uint8_t* img = image[it++ & 1];
                demote_tile<D, false, FMT>(rec8, img, kcode, vcode, lane_consts, k_scale, v_scale, sc, zp);
                uint4* out = reinterpret_cast<uint4*>(page3 + (size_t)m * TILE);
                for (int i = tid; i < TILE / 16; i += NT) out[i] = reinterpret_cast<const uint4*>(img)[i];
            }
        }
    }

    // copy-before-publish: every head's record is complete and visible before the id and tag appear.  The cluster
    // barrier (release / acquire) orders the record stores of every thread of the cluster before what the
    // publishing thread does next, and that thread's fence is cumulative: it orders them, device-wide, before its
    // own later stores.  (A fence in every thread would say the same and make each of them wait for its stores.)
    cluster_barrier();
    if (valid && crank == 0 && tid == 0 && entry_index != nullptr && (__threadfence(), last_cluster_of_page(page_tickets, page))) {
        const int64_t e = entry_index[page];
        if (e >= n_entries) atomicOr(status, kStBounds);      // an entry beyond the tables: flagged, nothing published
        else if (e >= 0) {
            block_table[e] = dst;
            __threadfence();
            tier_tag[e] = (uint8_t)MKV_TAG_STALE;
        }
    }
}

// Pages of several tiles, first pass of Demote: the minimum and maximum of every value channel over all tokens
// of the page, then the page's scale and zero (same arithmetic and order of the halves as in the 16-token
// record).  One cluster per (page, KV head); block r of the cluster scans tiles r, r + cluster size, ... with one
// thread per channel, the partial extremes meet in the first block through distributed shared memory.
// The extremes are defined by a scan in token order with strict comparisons; min/max instructions give the same
// value except for the sign of a zero extreme and a leading NaN, and those channels (rare) are scanned again
// literally, by the thread that writes the result.
__device__ __forceinline__ float ld_cluster_f32(const float* local, uint32_t rank)
{
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"((uint32_t)__cvta_generic_to_shared(local)), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

template <int D>
__global__ void __launch_bounds__(D) demote_minmax_kernel(const uint8_t* __restrict__ fp8, uint8_t* __restrict__ tq3,
                                                           int fp8_pages, int tq3_pages, int hkv, int tiles,
                                                           float v_scale, const int32_t* __restrict__ src_ids,
                                                           const int32_t* __restrict__ dst_ids)
{
    __shared__ float part[2][D];
    const int csize = (int)cluster_size(), crank = (int)cluster_rank();
    const int unit = blockIdx.x / csize, page = unit / hkv, h = unit % hkv, c = threadIdx.x;
    const int src = src_ids[page], dst = dst_ids[page];
    const bool valid = src >= 0 && src < fp8_pages && dst >= 0 && dst < tq3_pages;      // flagged by demote_kernel
    const uint8_t* page8 = fp8 + ((size_t)(valid ? src : 0) * hkv + h) * fp8_page_bytes(D, tiles);
    auto value = [&](uint32_t two, int half) {
        const float2 f = e4m3x2_to_f32(two & 0xFFFFu);
        return __fmul_rn(half ? f.y : f.x, v_scale);
    };
    // every block starts from the page's first token, so that a block without tiles is neutral
    const float first = valid ? value(*reinterpret_cast<const uint32_t*>(page8 + 16 * D + c * kPage), 0) : 0.f;
    float mn = first, mx = first;
    constexpr int AHEAD = 4;        // tiles whose loads are issued together (a thread's tiles are 4 KB apart)
    for (int m0 = crank; valid && m0 < tiles; m0 += AHEAD * csize) {
        uint4 raw[AHEAD];
#pragma unroll
        for (int u = 0; u < AHEAD; ++u) {
            const int m = m0 + u * csize;
            raw[u] = m < tiles ? *reinterpret_cast<const uint4*>(page8 + (size_t)m * fp8_record_bytes(D) + 16 * D + c * kPage)
                               : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < AHEAD; ++u) {
            if (m0 + u * csize >= tiles) break;
            const uint32_t rw[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
#pragma unroll
            for (int t = 0; t < kPage; t += 2) {
                const uint32_t two = rw[t >> 2] >> (8 * (t & 3));
                const float a = value(two, 0), b = value(two, 1);
                mn = fminf(mn, fminf(a, b));
                mx = fmaxf(mx, fmaxf(a, b));
            }
        }
    }
    part[0][c] = mn;
    part[1][c] = mx;
    cluster_barrier();
    if (crank == 0 && valid) {
        for (int k = 1; k < csize; ++k) {
            mn = fminf(mn, ld_cluster_f32(&part[0][c], (uint32_t)k));
            mx = fmaxf(mx, ld_cluster_f32(&part[1][c], (uint32_t)k));
        }
        if (!(mn != 0.0f && mx != 0.0f) || first != first) {
            // the literal scan: of equal values (+0 and -0) the earliest token counts
            mn = mx = first;
            for (int m = 0; m < tiles; ++m) {
                const uint4 raw = *reinterpret_cast<const uint4*>(page8 + (size_t)m * fp8_record_bytes(D) + 16 * D + c * kPage);
                const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                for (int t = 0; t < kPage; ++t) {
                    const float a = value(rw[t >> 2] >> (8 * (t & 2)), t & 1);
                    if (a < mn) mn = a;
                    if (a > mx) mx = a;
                }
            }
        }
        uint16_t* meta = reinterpret_cast<uint16_t*>(tq3 + ((size_t)dst * hkv + h) * tq3_page_bytes(D, tiles) +
                                                     (size_t)tiles * (12 * D + 32));
        const int cb = c >> 4, row = c & 15;
        const int hi = (cb >> 1) * 64 + (row & 7) * 8 + 4 * (cb & 1) + (row >> 3);
        meta[hi] = f32_to_f16_sat_bits(__fdiv_rn(__fsub_rn(mx, mn), 7.0f));
        meta[hi + 2] = f32_to_f16_sat_bits(mn);
    }
    cluster_barrier();              // the partial extremes stay readable until the first block has taken them
}

// Pages of several tiles, last pass of Demote / Promote: the kernels before it in the stream have written the
// whole page, so its id and tag may appear (copy-before-publish by stream order).
__global__ void publish_kernel(int n, const int32_t* __restrict__ src_ids, const int32_t* __restrict__ dst_ids,
                               int src_cap, int dst_cap, int32_t* block_table, uint8_t* tier_tag,
                               const int64_t* __restrict__ entry_index, int64_t n_entries, int tag, uint32_t* status)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int src = src_ids[i], dst = dst_ids[i];
    if (src < 0 || src >= src_cap || dst < 0 || dst >= dst_cap) return;
    const int64_t e = entry_index[i];
    if (e >= n_entries) atomicOr(status, kStBounds);
    else if (e >= 0) {
        block_table[e] = dst;
        __threadfence();
        tier_tag[e] = (uint8_t)tag;
    }
}

// Page tickets of the in-kernel publication: 48 counters in the pool's 256-byte status tail (word 0 is the status
// word, words 16..63 the tickets; the tail is zeroed with the arenas and every use leaves its counter at zero).
// Calls that convert more pages publish with a kernel of their own.
constexpr int kPageTickets = 48;
static uint32_t* page_tickets(mkv_pool* p) { return p->status_dev + 16; }

// grid rows of the tile-parallel passes: at least 16, and enough to fill the GPU when few pages are converted
static int tile_rows(int tiles, int n_pages, int hkv)
{
    int rows = (4 * 148 + n_pages * hkv - 1) / (n_pages * hkv);
    if (rows < 16) rows = 16;
    return rows < tiles ? rows : tiles;
}

template <typename Kernel, typename... Args>
static cudaError_t launch_clustered_rows(Kernel kernel, int n_pages, int csize, int rows, int threads, cudaStream_t s,
                                         Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_pages * csize, rows);
    cfg.blockDim = dim3(threads);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = csize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <int D, int FMT>
static int32_t launch_demote_d(mkv_pool* p, const int32_t* src, const int32_t* dst, int n, int32_t* bt, uint8_t* tags,
                               const int64_t* entry, int64_t n_entries, cudaStream_t s)
{
    const int c = heads_cluster(p->hkv, n);
    if (p->tiles == 1) {
        MKV_CUDA(launch_clustered(demote_kernel<D, false, FMT>, n, c, D, s, (const uint8_t*)p->fp8, p->tq3, p->cfg.fp8_pages,
                                  p->cfg.tq3_pages, p->hkv, 1, p->cfg.k_scale, p->cfg.v_scale, p->sigma, src, dst, bt,
                                  tags, entry, n_entries, p->status_dev, (uint32_t*)nullptr));
        return MKV_OK;
    }
    // pages of several tiles: scale/zero of the page, then the tiles in parallel, then the publication (from inside
    // the tile kernel when the call is small enough for the pool's page tickets, else as a kernel of its own)
    const bool fused = entry != nullptr && n <= kPageTickets;
    {
        // blocks per (page, head): up to a portable cluster of 8, fewer when the call fills the GPU anyway
        int cs = 8;
        while (cs > 1 && (cs > p->tiles || (long long)n * p->hkv * cs > 8LL * 148)) cs >>= 1;
        MKV_CUDA(launch_clustered(demote_minmax_kernel<D>, n * p->hkv, cs, D, s, (const uint8_t*)p->fp8, p->tq3, p->cfg.fp8_pages,
                                  p->cfg.tq3_pages, p->hkv, p->tiles, p->cfg.v_scale, src, dst));
    }
    MKV_CUDA(launch_clustered_rows(demote_kernel<D, true, FMT>, n, heads_cluster(p->hkv, 0), tile_rows(p->tiles, n, p->hkv), D, s,
                                   (const uint8_t*)p->fp8, p->tq3, p->cfg.fp8_pages, p->cfg.tq3_pages, p->hkv, p->tiles,
                                   p->cfg.k_scale, p->cfg.v_scale, p->sigma, src, dst, fused ? bt : (int32_t*)nullptr,
                                   fused ? tags : (uint8_t*)nullptr, fused ? entry : (const int64_t*)nullptr,
                                   fused ? n_entries : (int64_t)0, p->status_dev, fused ? page_tickets(p) : (uint32_t*)nullptr));
    if (entry && !fused) {
        publish_kernel<<<(n + 127) / 128, 128, 0, s>>>(n, src, dst, p->cfg.fp8_pages, p->cfg.tq3_pages, bt, tags, entry,
                                                       n_entries, MKV_TAG_STALE, p->status_dev);
        MKV_CUDA(cudaGetLastError());
    }
    (void)c;
    return MKV_OK;
}

int32_t launch_demote(mkv_pool* p, const int32_t* src, const int32_t* dst, int n, int32_t* bt, uint8_t* tags,
                      const int64_t* entry, int64_t n_entries, cudaStream_t s)
{
    if (p->fmt == 2)
        return p->d == 128 ? launch_demote_d<128, 2>(p, src, dst, n, bt, tags, entry, n_entries, s)
                           : launch_demote_d<256, 2>(p, src, dst, n, bt, tags, entry, n_entries, s);
    return p->d == 128 ? launch_demote_d<128, 1>(p, src, dst, n, bt, tags, entry, n_entries, s)
                       : launch_demote_d<256, 1>(p, src, dst, n, bt, tags, entry, n_entries, s);
}

// ------------------------------------------------------------------------------------------ promote
// Promote (Algorithm 1 step 3): reconstruct a Stale page into a newly allocated FP8 page, then publish
// it as Anchor.  One cluster per page, its blocks sharing out the KV heads as in demote_kernel.  The
// record is staged in shared memory;
// warps rebuild key vectors (signed levels, shuffle Walsh-Hadamard, norm correction, sign), threads
// rebuild value channels; the fp32 operation order is fixed so that the written bytes are reproducible.
//
// Reading the code sections back (inverse of the packer in demote_kernel): fragment lane
// L = 4 (row % 8) + (slot % 8) / 2 holds, in nibble 2 rr + slot % 2 with rr = row / 8 + 2 (slot / 8),
// the entry (row, slot) of every 16 x 16 block; for keys row = token and slot = channel % 16, for
// values row = channel % 16 and slot = token.
// D = A B + C with 8-bit integers: A 16 x 32 (row-major fragments), B 32 x 8 (column-major), C 16 x 8 in int32
__device__ __forceinline__ void imma16832(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Keys of one record of format 2 back to e4m3 rows (Promote), the inverse rotation as a matrix product.
// The levels of format 2 are eighths of the integers +-2, +-6, +-11, +-18, so the transform H c of a token's d
// levels consists of sums of integers below 2^13: every order of summation gives the same value, and the
// butterflies can be replaced by the product C[16 tokens x d] H[d x d] in 8-bit integer tensor-core
// instructions (exact int32 sums).  The record's key section already is the A operand: lane 4 (t % 8) + (k % 16) / 4
// holds, per 32-dim step, the codes of tokens g, g + 8 at dims 4 tq .. + 3 and 16 + 4 tq .. + 3, and one
// byte-table lookup turns four codes into four signed bytes.  H[k][n] = (-1)^popcount(k & n) needs no table: for
// lane (g, tq), column n = 8 j + g and rows k = 32 s + 16 b + 4 tq + i its sign is the product of a per-lane
// pattern over i, a per-warp part and a part that is known at compile time.
// Warp w computes the column tiles j = w, w + D/32, ... (eight columns each); results go to `ktile`
// [16 tokens][D] e4m3 in shared memory.  All D threads call it; the caller synchronises before reading ktile.
// What promote_keys_v2 needs per lane and warp, computed once per block.
template <int D>
struct PromoteKeyLane {
    uint32_t b0p, b1p, b0n, b1n;          // B fragments of H for this lane: both K halves, plain and negated
    uint32_t o0p, o1p, o0n, o1n;          // the same for the odd steps (negated in warps whose columns have bit 5 of n set)
    uint32_t flip[D / 8 / (D / 32)][2];   // rotation signs of the lane's two columns of every tile, as fp32 sign bits
    __device__ __forceinline__ void init(const SigmaBits& sigma, int warp, int lane)
    {
        constexpr uint32_t NEG = 0xFEFEFEFEu;             // x ^ NEG negates bytes +-1
        constexpr int NWARP = D / 32, NTILE = D / 8 / NWARP;
        const int g = lane >> 2, tq = lane & 3;
        // (-1)^popcount(k & n), k = 32 s + 16 b + 4 tq + i, n = 8 j + g, j = NWARP t + warp:
        //   bits 0-1: i & g -> the byte pattern W over i;  bit 2: tq0 & g2;  bit 3: tq1 & j0 (j0 = warp & 1);
        //   bit 4: b & j1 (j1 = (warp >> 1) & 1);  bits 5-7: s & (j >> 2), of which bit 0 of j >> 2 is warp >> 2 for
        //   D = 256 (it negates the odd steps) and the rest is the tile index (compile time)
        const uint32_t W = (g & 3) == 0 ? 0x01010101u : (g & 3) == 1 ? 0xFF01FF01u : (g & 3) == 2 ? 0xFFFF0101u : 0x01FFFF01u;
        const bool lane_odd = (((tq & 1) & (g >> 2)) ^ ((tq >> 1) & (warp & 1))) != 0;
        b0p = lane_odd ? (W ^ NEG) : W;
        b1p = ((warp >> 1) & 1) ? (b0p ^ NEG) : b0p;
        b0n = b0p ^ NEG;
        b1n = b1p ^ NEG;
        const bool w2 = ((warp >> 2) & 1) != 0;
        o0p = w2 ? b0n : b0p;
        o1p = w2 ? b1n : b1p;
        o0n = w2 ? b0p : b0n;
        o1n = w2 ? b1p : b1n;
#pragma unroll
        for (int t = 0; t < NTILE; ++t) {
            const int n0 = 8 * (NWARP * t + warp) + 2 * tq;
            const uint32_t sg = (sigma.w[n0 >> 5] >> (n0 & 31)) & 3u;
            flip[t][0] = (sg & 1u) << 31;
            flip[t][1] = (sg & 2u) << 30;
        }
    }
};

// Keys of one record of format 2 back to e4m3 rows (Promote), the inverse rotation as a matrix product.
// The levels of format 2 are eighths of the integers +-2, +-6, +-11, +-18, so the transform H c of a token's d
// levels consists of sums of integers below 2^13: every order of summation gives the same value, and the
// butterflies can be replaced by the product C[16 tokens x d] H[d x d] in 8-bit integer tensor-core
// instructions (exact int32 sums).  The record's key section already is the A operand: lane 4 (t % 8) + (k % 16) / 4
// holds, per 32-dim step, the codes of tokens g, g + 8 at dims 4 tq .. + 3 and 16 + 4 tq .. + 3, and one
// byte-table lookup turns four codes into four signed bytes.  H[k][n] = (-1)^popcount(k & n) needs no table
// (PromoteKeyLane).  Warp w computes the column tiles j = w, w + D/32, ... (eight columns each); results go to
// `ktile` [16 tokens][D] e4m3 in shared memory.  All D threads call it; the caller synchronises before reading ktile.
template <int D>
__device__ __forceinline__ void promote_keys_v2(const uint8_t* img, uint8_t* ktile, uint4* afrag, const PromoteKeyLane<D>& L,
                                                float rs, float inv_k_scale, bool unit_k)
{
    constexpr int NS = D / 32;            // 32-dim steps (K of the product)
    constexpr int NWARP = D / 32;         // warps of the block
    constexpr int NTILE = D / 8 / NWARP;  // column tiles per warp (4)
    constexpr uint32_t T0 = 0x120B0602u, T1 = 0xEEF5FAFEu;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    // ---- A: the record's codes as signed bytes, 4 registers per step.  Warp s unpacks step s for everybody
    // (afrag [step][lane] in shared memory), then every warp fetches all steps.
    {
        const int j = warp >> 1;
        const uint32_t A = *reinterpret_cast<const uint32_t*>(img + lane_word_offset(D, lane, 3 * j));
        const uint32_t Bw = *reinterpret_cast<const uint32_t*>(img + lane_word_offset(D, lane, 3 * j + 1));
        const uint32_t Cw = *reinterpret_cast<const uint32_t*>(img + lane_word_offset(D, lane, 3 * j + 2));
        uint32_t s0, s1;
        if ((warp & 1) == 0) {
            s0 = A & 0x77777777u;
            s1 = Bw & 0x77777777u;
        } else {
            s0 = ((A >> 1) & 0x44444444u) | (Cw & 0x33333333u);
            s1 = ((Bw >> 1) & 0x44444444u) | ((Cw >> 2) & 0x33333333u);
        }
        uint4 v;
        v.x = __byte_perm(T0, T1, s0);            // token g, dims 4 tq ..
        v.z = __byte_perm(T0, T1, s0 >> 16);      // token g, dims 16 + 4 tq ..
        v.y = __byte_perm(T0, T1, s1);            // token g + 8
        v.w = __byte_perm(T0, T1, s1 >> 16);
        afrag[warp * 32 + lane] = v;
    }
    __syncthreads();
    uint32_t a[NS][4];
#pragma unroll
    for (int s_ = 0; s_ < NS; ++s_) {
        const uint4 v = afrag[s_ * 32 + lane];
        a[s_][0] = v.x; a[s_][1] = v.y; a[s_][2] = v.z; a[s_][3] = v.w;
    }
    // ---- per token scale g r / 8
    const __half* gh = reinterpret_cast<const __half*>(img + 12 * D);
    const float gr0 = __fmul_rn(__fmul_rn(__half2float(gh[g]), rs), 0.125f);
    const float gr1 = __fmul_rn(__fmul_rn(__half2float(gh[g + 8]), rs), 0.125f);
    float out[NTILE][4];
#pragma unroll
    for (int t = 0; t < NTILE; ++t) {
        constexpr int JH = NWARP / 4;                     // j >> 2 = JH * t + (warp >> 2)
        int c[4] = {0, 0, 0, 0};
#pragma unroll
        for (int s_ = 0; s_ < NS; ++s_) {
            const bool neg = (__popc((unsigned)(s_ & (JH * t) & (NWARP == 8 ? 6 : 7))) & 1) != 0;     // compile-time part of bits 5-7
            if (s_ & 1) imma16832(c, a[s_][0], a[s_][1], a[s_][2], a[s_][3], neg ? L.o0n : L.o0p, neg ? L.o1n : L.o1p);
            else imma16832(c, a[s_][0], a[s_][1], a[s_][2], a[s_][3], neg ? L.b0n : L.b0p, neg ? L.b1n : L.b1p);
        }
        // columns n = 8 j + 2 tq, + 1 of tokens g (c0, c1) and g + 8 (c2, c3); j = NWARP t + warp
        out[t][0] = __uint_as_float(__float_as_uint(__fmul_rn(gr0, (float)c[0])) ^ L.flip[t][0]);
        out[t][1] = __uint_as_float(__float_as_uint(__fmul_rn(gr0, (float)c[1])) ^ L.flip[t][1]);
        out[t][2] = __uint_as_float(__float_as_uint(__fmul_rn(gr1, (float)c[2])) ^ L.flip[t][0]);
        out[t][3] = __uint_as_float(__float_as_uint(__fmul_rn(gr1, (float)c[3])) ^ L.flip[t][1]);
    }
    if (!unit_k) {                        // a product with 1 is skipped (a branch, not predicated multiplications)
#pragma unroll
        for (int t = 0; t < NTILE; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) out[t][e] = __fmul_rn(out[t][e], inv_k_scale);
    }
#pragma unroll
    for (int t = 0; t < NTILE; ++t) {
        const int n0 = 8 * (NWARP * t + warp) + 2 * tq;
        *reinterpret_cast<uint16_t*>(ktile + g * D + n0) =
            (uint16_t)__nv_cvt_float2_to_fp8x2(make_float2(out[t][0], out[t][1]), __NV_SATFINITE, __NV_E4M3);
        *reinterpret_cast<uint16_t*>(ktile + (g + 8) * D + n0) =
            (uint16_t)__nv_cvt_float2_to_fp8x2(make_float2(out[t][2], out[t][3]), __NV_SATFINITE, __NV_E4M3);
    }
}

template <int D, bool BIG, int FMT>
__global__ void __launch_bounds__(D) promote_kernel(const uint8_t* __restrict__ tq3, uint8_t* __restrict__ fp8,
                                                     int tq3_pages, int fp8_pages, int hkv, int tiles, float inv_k_scale,
                                                     float inv_v_scale, float rs, SigmaBits sigma,
                                                     const int32_t* __restrict__ src_ids,
                                                     const int32_t* __restrict__ dst_ids, int32_t* block_table,
                                                     uint8_t* tier_tag, const int64_t* entry_index, int64_t n_entries,
                                                     uint32_t* __restrict__ status, uint32_t* page_tickets)
{
    constexpr int EPL = D / 32;
    constexpr int NT = D;
    constexpr int REC = 16 * D + 32;
    __shared__ __align__(16) uint8_t image[2][REC];
    __shared__ __align__(16) uint8_t ktile[FMT == 2 ? kPage * D : 16];   // format 2: the rebuilt key rows of one record
    __shared__ uint4 afrag[FMT == 2 ? D : 1];                            // format 2: [32-dim step][lane] A operands of the key product
    __shared__ float level[8];            // signed key levels by 3-bit code

    const int csize = (int)cluster_size(), crank = (int)cluster_rank();
    const int page = blockIdx.x / csize, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int src = src_ids[page], dst = dst_ids[page];
    const bool valid = src >= 0 && src < tq3_pages && dst >= 0 && dst < fp8_pages;
    if (!valid && tid == 0 && crank == 0 && blockIdx.y == 0) atomicOr(status, kStBounds);
    if (tid < 8) {
        using CB = KeyCodebook<FMT>;
        const float c = (tid & 3) == 0 ? CB::C0 : (tid & 3) == 1 ? CB::C1 : (tid & 3) == 2 ? CB::C2 : CB::C3;
        level[tid] = (tid & 4) ? -c : c;
    }
    // ---- per-lane constants of the key path: this lane rebuilds channels lane*EPL .. +EPL-1
    const int kb = (lane * EPL) >> 4, s0 = (lane * EPL) & 15;       // 16-channel block, first slot in it
    const int kj = kb >> 2, kind = kb & 3;
    const int w_sgn = 3 * kj + (kind & 1);                          // word A or B: codes of kinds 0/1, signs of 2/3
    const int w_mag = kind < 2 ? w_sgn : 3 * kj + 2;                // word C holds the magnitudes of kinds 2/3
    const int off_sgn = lane_word_offset(D, 0, w_sgn), off_mag = lane_word_offset(D, 0, w_mag);
    const int str_sgn = lane_word_offset(D, 1, w_sgn) - off_sgn, str_mag = lane_word_offset(D, 1, w_mag) - off_mag;
    const int mag_extra = kind == 3 ? 2 : 0;                        // high pair of the C nibble
    const uint32_t mag_mask = kind < 2 ? 7u : 3u;                   // kinds 0/1 read sign and magnitude at once
    const uint32_t sgn_mask = kind < 2 ? 0u : 4u;
    uint32_t flip[EPL];
#pragma unroll
    for (int r = 0; r < EPL; ++r) {
        const int i = lane * EPL + r;
        flip[r] = ((sigma.w[i >> 5] >> (i & 31)) & 1u) << 31;
    }
    float sgn[5];                           // butterfly stage b: lanes with bit b set subtract
#pragma unroll
    for (int b = 0; b < 5; ++b) sgn[b] = ((lane >> b) & 1) ? -1.0f : 1.0f;
    const bool unit_k = inv_k_scale == 1.0f, unit_v = inv_v_scale == 1.0f;   // a product with 1 is skipped
    PromoteKeyLane<D> key_lane;
    if constexpr (FMT == 2) key_lane.init(sigma, warp, lane);
    // ---- per-thread constants of the value path: this thread rebuilds channel tid
    const int cb = tid >> 4, row = tid & 15;
    const int vj = cb >> 2, grp = (cb & 3) >> 1, k0 = 4 * (cb & 1) + (row >> 3);
    const int off_v = 6 * D + lane_word_offset(D, 4 * (row & 7), 3 * vj + grp);
    const int off_v1 = 6 * D + lane_word_offset(D, 4 * (row & 7), 3 * vj + grp + 1);
    const int str_v = lane_word_offset(D, 1, 3 * vj + grp) - lane_word_offset(D, 0, 3 * vj + grp);
    const int str_v1 = lane_word_offset(D, 1, 3 * vj + grp + 1) - lane_word_offset(D, 0, 3 * vj + grp + 1);
    const uint32_t sel0 = grp == 0 ? 0x0410u : 0x0541u, sel1 = grp == 0 ? 0x0632u : 0x0763u;
    const int meta_i = (cb >> 1) * 64 + (row & 7) * 8 + 4 * (cb & 1) + (row >> 3);

    // 16-token pages: one record per head.  Pages of several tiles: the blocks of grid row y take tiles y,
    // y + gridDim.y, ...; a tile and the page's scale/zero behind it form the same image as a 16-token record.
    constexpr int TILE = 12 * D + 32;
    const int m_first = BIG ? (int)blockIdx.y : 0, m_step = BIG ? (int)gridDim.y : 1, m_end = BIG ? tiles : 1;
    // The record of the next (head, tile) is copied into the other image asynchronously while this one is rebuilt.
    auto fetch = [&](int h, int m, uint8_t* img) {
        const uint8_t* page3 = tq3 + ((size_t)src * hkv + h) * tq3_page_bytes(D, tiles);
        const uint8_t* rec3 = page3 + (size_t)m * TILE;
        if constexpr (!BIG) {
            for (int i = tid; i < REC / 16; i += NT) cp_async16(img + 16 * i, rec3 + 16 * i);
        } else {
            const uint8_t* meta = page3 + (size_t)tiles * TILE;
            for (int i = tid; i < TILE / 16; i += NT) cp_async16(img + 16 * i, rec3 + 16 * i);
            for (int i = tid; i < 4 * D / 16; i += NT) cp_async16(img + TILE + 16 * i, meta + 16 * i);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    int h = crank, m = m_first;
    bool more = valid && h < hkv && m < m_end;
    if (more) fetch(h, m, image[0]);
    for (int it = 0; more; ++it) {
        int hn = h, mn = m + m_step;
        if (mn >= m_end) {
            mn = m_first;
            hn = h + csize;
        }
        const bool more_next = hn < hkv;
        uint8_t* rec8 = fp8 + (((size_t)dst * hkv + h) * tiles + m) * fp8_record_bytes(D);
        uint8_t* img = image[it & 1];
        asm volatile("cp.async.wait_all;" ::: "memory");
        __syncthreads();            // this image has landed for every thread; the other image and ktile are no longer read
        if (more_next) fetch(hn, mn, image[(it + 1) & 1]);

        // ---- keys.  Format 2: the inverse rotation as an integer matrix product (all warps, every token at once)
        if constexpr (FMT == 2) promote_keys_v2<D>(img, ktile, afrag, key_lane, rs, inv_k_scale, unit_k);
        // Format 1: warp w rebuilds tokens w, w + NT/32, ... with butterflies
        for (int tok = warp; FMT != 2 && tok < kPage; tok += NT / 32) {
            float y[EPL];
            if constexpr (FMT == 2) {
                // record format 2: four consecutive dims are the nibbles of one half-word of register
                // e = 4 (step % 2) + 2 (token / 8) + (k / 16) in the triple step / 2 of fragment lane 4 (token % 8) + (k % 16) / 4
#pragma unroll
                for (int gi = 0; gi < EPL / 4; ++gi) {
                    const int i0 = lane * EPL + 4 * gi, st = i0 >> 5, k = i0 & 31, j = st >> 1;
                    const int e = 4 * (st & 1) + 2 * (tok >> 3) + (k >> 4), L = 4 * (tok & 7) + ((k & 15) >> 2), sh = 16 * (e & 1);
                    const uint32_t A = *reinterpret_cast<const uint32_t*>(img + lane_word_offset(D, L, 3 * j));
                    const uint32_t Bw = *reinterpret_cast<const uint32_t*>(img + lane_word_offset(D, L, 3 * j + 1));
                    const uint32_t Cw = *reinterpret_cast<const uint32_t*>(img + lane_word_offset(D, L, 3 * j + 2));
                    uint32_t nib;
                    if (e < 2) nib = (A >> sh) & 0x7777u;
                    else if (e < 4) nib = (Bw >> sh) & 0x7777u;
                    else if (e < 6) nib = ((Cw >> sh) & 0x3333u) | ((A >> (sh + 1)) & 0x4444u);
                    else nib = ((Cw >> (sh + 2)) & 0x3333u) | ((Bw >> (sh + 1)) & 0x4444u);
                    // one byte-table lookup for the four codes: 8 x the signed level (2, 6, 11, 18 | negated).  The
                    // transform below is exact on these integers, so the factor 1/8 moves into the token's scale
                    const uint32_t lv = __byte_perm(0x120B0602u, 0xEEF5FAFEu, nib);
#pragma unroll
                    for (int x = 0; x < 4; ++x) y[4 * gi + x] = (float)(int)(int8_t)(lv >> (8 * x));
                }
            }
#pragma unroll
            for (int r2 = 0; r2 < (FMT == 2 ? 0 : EPL); r2 += 2) {
                const int s = s0 + r2;                                    // even slot; s + 1 shares the word
                const int L = 4 * (tok & 7) + ((s & 7) >> 1), n = 2 * ((tok >> 3) + 2 * (s >> 3));
                const uint32_t ws = *reinterpret_cast<const uint32_t*>(img + off_sgn + L * str_sgn) >> (4 * n);
                const uint32_t wm = *reinterpret_cast<const uint32_t*>(img + off_mag + L * str_mag) >> (4 * n + mag_extra);
                const uint32_t c_even = (wm & mag_mask) | ((ws >> 1) & sgn_mask);
                const uint32_t c_odd = ((wm >> 4) & mag_mask) | ((ws >> 5) & sgn_mask);
                y[r2] = level[c_even];
                y[r2 + 1] = level[c_odd];
            }
#pragma unroll
            for (int hh = 1; hh < EPL; hh <<= 1)
#pragma unroll
                for (int r = 0; r < EPL; ++r)
                    if ((r & hh) == 0) {
                        const float u = y[r], w = y[r + hh];
                        y[r] = __fadd_rn(u, w);
                        y[r + hh] = __fsub_rn(u, w);
                    }
#pragma unroll
            for (int b = 0; b < 5; ++b)
#pragma unroll
                for (int r = 0; r < EPL; ++r) {
                    // o + y or o - y: the product with +-1 is exact, one rounding as in the single addition
                    const float o = __shfl_xor_sync(0xffffffffu, y[r], 1 << b);
                    y[r] = __fmaf_rn(y[r], sgn[b], o);
                }
            const float g = __half2float(reinterpret_cast<const __half*>(img + 12 * D)[tok]);
            // format 2: y holds 8 x the transform of the levels (all sums of the transform are exact integers below
            // 2^13, so H(8 c) = 8 H(c) bit for bit) and gr y = (gr / 8)(8 y) is the same real product, rounded once
            const float gr = FMT == 2 ? __fmul_rn(__fmul_rn(g, rs), 0.125f) : __fmul_rn(g, rs);
            uint32_t out[EPL / 4];
#pragma unroll
            for (int r = 0; r < EPL / 4; ++r) out[r] = 0;
#pragma unroll
            for (int r = 0; r < EPL; r += 2) {
                float2 kk;
                kk.x = __uint_as_float(__float_as_uint(__fmul_rn(gr, y[r])) ^ flip[r]);
                kk.y = __uint_as_float(__float_as_uint(__fmul_rn(gr, y[r + 1])) ^ flip[r + 1]);
                if (!unit_k) {
                    kk.x = __fmul_rn(kk.x, inv_k_scale);
                    kk.y = __fmul_rn(kk.y, inv_k_scale);
                }
                out[r >> 2] |= (uint32_t)__nv_cvt_float2_to_fp8x2(kk, __NV_SATFINITE, __NV_E4M3) << (8 * (r & 3));
            }
            if constexpr (EPL == 8)
                *reinterpret_cast<uint2*>(rec8 + tok * D + lane * EPL) = make_uint2(out[0], out[1]);
            else
                *reinterpret_cast<uint32_t*>(rec8 + tok * D + lane * EPL) = out[0];
        }
        // ---- values: one thread per channel; fragment lane 4 (row % 8) + q holds tokens 2q, 2q+1, 2q+8, 2q+9
        {
            const __half* meta = reinterpret_cast<const __half*>(img + 12 * D + 32);
            const float sc = __half2float(meta[meta_i]), zp = __half2float(meta[meta_i + 2]);
            // The channel's eight possible output bytes, e4m3((sc * code + zp) / v_scale) for code 0..7, computed
            // once; a byte-table lookup then turns the codes of four tokens into four output bytes.
            float lv[8];
#pragma unroll
            for (int cde = 0; cde < 8; ++cde) lv[cde] = __fadd_rn(__fmul_rn(sc, (float)cde), zp);
            if (!unit_v) {
#pragma unroll
                for (int cde = 0; cde < 8; ++cde) lv[cde] = __fmul_rn(lv[cde], inv_v_scale);
            }
            uint32_t pr[4];
#pragma unroll
            for (int cde = 0; cde < 8; cde += 2)
                pr[cde >> 1] = (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(lv[cde], lv[cde + 1]), __NV_SATFINITE, __NV_E4M3);
            const uint32_t lut_lo = pr[0] | (pr[1] << 16), lut_hi = pr[2] | (pr[3] << 16);
            uint32_t near[4], far[4];           // per q: codes of tokens (2q, 2q+1) and (2q+8, 2q+9) as two nibbles
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t lo = *reinterpret_cast<const uint32_t*>(img + off_v + q * str_v);
                const uint32_t hi = *reinterpret_cast<const uint32_t*>(img + off_v1 + q * str_v1);
                const uint32_t st0 = __byte_perm(lo, hi, sel0) >> (3 * k0);          // stream of the even tokens
                const uint32_t st1 = __byte_perm(lo, hi, sel1) >> (3 * k0);          // stream of the odd tokens
                near[q] = (st0 & 7u) | ((st1 & 7u) << 4);
                far[q] = ((st0 >> 6) & 7u) | (((st1 >> 6) & 7u) << 4);
            }
            uint32_t out[4];
            out[0] = __byte_perm(lut_lo, lut_hi, near[0] | (near[1] << 8));           // tokens 0..3
            out[1] = __byte_perm(lut_lo, lut_hi, near[2] | (near[3] << 8));           // tokens 4..7
            out[2] = __byte_perm(lut_lo, lut_hi, far[0] | (far[1] << 8));             // tokens 8..11
            out[3] = __byte_perm(lut_lo, lut_hi, far[2] | (far[3] << 8));             // tokens 12..15
            *reinterpret_cast<uint4*>(rec8 + 16 * D + tid * kPage) = make_uint4(out[0], out[1], out[2], out[3]);
        }
        if constexpr (FMT == 2) {
            __syncthreads();               // key rows complete; the next record's rows are written after the next barrier
            reinterpret_cast<uint4*>(rec8)[tid] = reinterpret_cast<const uint4*>(ktile)[tid];      // 16 D bytes, D threads
        }
        h = hn;
        m = mn;
        more = more_next;
    }
    // copy-before-publish (as in demote_kernel: cluster barrier, then the publishing thread's cumulative fence)
    cluster_barrier();
    if (valid && crank == 0 && tid == 0 && entry_index != nullptr && (__threadfence(), last_cluster_of_page(page_tickets, page))) {
        const int64_t e = entry_index[page];
        if (e >= n_entries) atomicOr(status, kStBounds);
        else if (e >= 0) {
            block_table[e] = dst;
            __threadfence();
            tier_tag[e] = (uint8_t)MKV_TAG_ANCHOR;
        }
    }
}

template <int D, int FMT>
static int32_t launch_promote_d(mkv_pool* p, const int32_t* src, const int32_t* dst, int n, int32_t* bt, uint8_t* tags,
                                const int64_t* entry, int64_t n_entries, cudaStream_t s)
{
    const float ik = 1.0f / p->cfg.k_scale, iv = 1.0f / p->cfg.v_scale;
    const float rs = (float)(1.0 / sqrt((double)p->d));
    if (p->tiles == 1) {
        MKV_CUDA(launch_clustered(promote_kernel<D, false, FMT>, n, heads_cluster(p->hkv, n), D, s, (const uint8_t*)p->tq3, p->fp8,
                                  p->cfg.tq3_pages, p->cfg.fp8_pages, p->hkv, 1, ik, iv, rs, p->sigma, src, dst, bt, tags,
                                  entry, n_entries, p->status_dev, (uint32_t*)nullptr));
        return MKV_OK;
    }
    const bool fused = entry != nullptr && n <= kPageTickets;
    MKV_CUDA(launch_clustered_rows(promote_kernel<D, true, FMT>, n, heads_cluster(p->hkv, 0), tile_rows(p->tiles, n, p->hkv), D, s,
                                   (const uint8_t*)p->tq3, p->fp8, p->cfg.tq3_pages, p->cfg.fp8_pages, p->hkv, p->tiles, ik,
                                   iv, rs, p->sigma, src, dst, fused ? bt : (int32_t*)nullptr, fused ? tags : (uint8_t*)nullptr,
                                   fused ? entry : (const int64_t*)nullptr, fused ? n_entries : (int64_t)0, p->status_dev,
                                   fused ? page_tickets(p) : (uint32_t*)nullptr));
    if (entry && !fused) {
        publish_kernel<<<(n + 127) / 128, 128, 0, s>>>(n, src, dst, p->cfg.tq3_pages, p->cfg.fp8_pages, bt, tags, entry,
                                                       n_entries, MKV_TAG_ANCHOR, p->status_dev);
        MKV_CUDA(cudaGetLastError());
    }
    return MKV_OK;
}

int32_t launch_promote(mkv_pool* p, const int32_t* src, const int32_t* dst, int n, int32_t* bt, uint8_t* tags,
                       const int64_t* entry, int64_t n_entries, cudaStream_t s)
{
    if (p->fmt == 2)
        return p->d == 128 ? launch_promote_d<128, 2>(p, src, dst, n, bt, tags, entry, n_entries, s)
                           : launch_promote_d<256, 2>(p, src, dst, n, bt, tags, entry, n_entries, s);
    return p->d == 128 ? launch_promote_d<128, 1>(p, src, dst, n, bt, tags, entry, n_entries, s)
                       : launch_promote_d<256, 1>(p, src, dst, n, bt, tags, entry, n_entries, s);
}

// ------------------------------------------------------------------------------------------ anchor
__global__ void set_anchor_kernel(uint8_t* tags, int64_t entry, int flag, uint32_t* status)
{
    if (tags[entry] == MKV_TAG_STALE)
        atomicOr(status, kStState);
    else
        tags[entry] = flag ? MKV_TAG_ANCHOR : MKV_TAG_RECENT;
}

int32_t launch_set_anchor(mkv_pool* p, uint8_t* tags, int64_t entry, int flag, cudaStream_t s)
{
    set_anchor_kernel<<<1, 1, 0, s>>>(tags, entry, flag, p->status_dev);
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
}

}  // namespace mkv
