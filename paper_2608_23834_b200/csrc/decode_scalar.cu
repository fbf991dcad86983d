// CUDA-core decode attention (MKV_DECODE_SCALAR): the same one-pass mixed-format split-KV scan as
// the tensor-core kernel, written with plain fp32 FMAs and a generic bit-by-bit TQ3 unpack.  It is
// the measured alternative that justifies the tensor-core kernel, and a second implementation of
// the record layout.  Section 3.3 (per-partition m, l, O and Eq. softmax-merge), Section 4.1.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <math_constants.h>

#include "mkv_internal.cuh"

namespace mkv {

int scalar_splits(int B, int hkv)
{
    int s = 592 / (B * hkv);
    return s < 1 ? 1 : (s > 64 ? 64 : s);
}

size_t decode_ws_scalar_bytes(int B, int hkv, int group, int d)
{
    return (size_t)B * hkv * group * scalar_splits(B, hkv) * (d + 2) * sizeof(float);
}

__device__ __forceinline__ float e4m3_f32(uint8_t b)
{
    __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)b, __NV_E4M3);
    return __half2float(__half(h));
}

template <int D>
__device__ __forceinline__ uint32_t lane_word(const uint8_t* section, int lane, int w)
{
    return *reinterpret_cast<const uint32_t*>(section + lane_word_offset(D, lane, w));
}

// 3-bit key code of (token t, rotated dim i): magnitude in bits 0-1, sign in bit 2
template <int D>
__device__ int tq3_key_code(const uint8_t* rec, int t, int i, int fmt)
{
    if (fmt == 2) {
        // record format 2: step i/32, K slot k = i%32; lane 4 (t%8) + (k%16)/4, register e = 4 (step%2) + 2 (t/8) + k/16
        // of word triple step/2, nibble 4 (e%2) + k%4
        const int st = i >> 5, k = i & 31;
        const int lane = 4 * (t & 7) + ((k & 15) >> 2), j = st >> 1, e = 4 * (st & 1) + 2 * (t >> 3) + (k >> 4);
        const int n = 4 * (e & 1) + (k & 3);
        const uint32_t A = lane_word<D>(rec, lane, 3 * j), Bw = lane_word<D>(rec, lane, 3 * j + 1),
                       Cw = lane_word<D>(rec, lane, 3 * j + 2);
        if (e < 2) return (A >> (4 * n)) & 7;
        if (e < 4) return (Bw >> (4 * n)) & 7;
        if (e < 6) return ((Cw >> (4 * n)) & 3) | (((A >> (4 * n + 3)) & 1) << 2);
        return ((Cw >> (4 * n + 2)) & 3) | (((Bw >> (4 * n + 3)) & 1) << 2);
    }
    const int kb = i >> 4, s = i & 15;
    const int lane = 4 * (t & 7) + ((s & 7) >> 1), r = (t >> 3) + 2 * (s >> 3), n = 2 * r + (s & 1), j = kb >> 2;
    const uint32_t A = lane_word<D>(rec, lane, 3 * j), Bw = lane_word<D>(rec, lane, 3 * j + 1),
                   Cw = lane_word<D>(rec, lane, 3 * j + 2);
    switch (kb & 3) {
    case 0: return (A >> (4 * n)) & 7;
    case 1: return (Bw >> (4 * n)) & 7;
    case 2: return ((Cw >> (4 * n)) & 3) | (((A >> (4 * n + 3)) & 1) << 2);
    default: return ((Cw >> (4 * n + 2)) & 3) | (((Bw >> (4 * n + 3)) & 1) << 2);
    }
}

// 3-bit value code of (token t, channel c)
template <int D>
__device__ int tq3_value_code(const uint8_t* rec, int t, int c)
{
    const int cb = c >> 4, row = c & 15;
    const int lane = 4 * (row & 7) + ((t & 7) >> 1), r = (row >> 3) + 2 * (t >> 3), half = t & 1;
    const int j = cb >> 2, grp = (cb & 3) >> 1, k = 4 * (cb & 1) + r;
    const uint8_t* sec = rec + 6 * D;
    const uint32_t W0 = lane_word<D>(sec, lane, 3 * j), W1 = lane_word<D>(sec, lane, 3 * j + 1),
                   W2 = lane_word<D>(sec, lane, 3 * j + 2);
    auto by = [](uint32_t w, int b) { return (w >> (8 * b)) & 0xFFu; };
    uint32_t st;
    if (grp == 0)
        st = half == 0 ? (by(W0, 0) | by(W0, 1) << 8 | by(W1, 0) << 16) : (by(W0, 2) | by(W0, 3) << 8 | by(W1, 2) << 16);
    else
        st = half == 0 ? (by(W1, 1) | by(W2, 0) << 8 | by(W2, 1) << 16) : (by(W1, 3) | by(W2, 2) << 8 | by(W2, 3) << 16);
    return (st >> (3 * k)) & 7;
}

template <int D>
__global__ void __launch_bounds__(D) decode_scalar_kernel(
    const uint8_t* __restrict__ fp8, const uint8_t* __restrict__ tq3, int fp8_pages, int tq3_pages, int hkv, int G,
    float k_scale, float v_scale, SigmaBits sigma, const __nv_bfloat16* __restrict__ q,
    const int32_t* __restrict__ bt, const uint8_t* __restrict__ tags, const int32_t* __restrict__ lens,
    int max_pages, int tiles, int fmt, float scale, int n_splits, float* __restrict__ part, uint32_t* __restrict__ status)
{
    extern __shared__ float smem[];
    float* qs = smem;                       // [8][D] query
    float* qr = qs + 8 * D;                 // [8][D] rotated query  q' = d^-1/2 H (sigma . q)
    float* Ks = qr + 8 * D;                 // [16][D+1] dequantised keys (TQ3: signed centroids, rotated domain)
    float* Vs = Ks + kPage * (D + 1);       // [16][D]
    float* red = Vs + kPage * D;            // [2][128] partial dot products
    float* sc = red + 256;                  // [16][8] scores
    float* gn = sc + 128;                   // [16] norm corrections
    const int tid = threadIdx.x, split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int hq = hkv * G;
    // a length beyond the table row is cut to the row and flagged, so that no entry past it is read
    const long long cap = (long long)max_pages * tiles * kPage;
    int len = lens[b];
    if (len > cap) {
        if (tid == 0) atomicOr(status, kStBounds);
        len = (int)cap;
    }
    if (len < 0) len = 0;
    const int n_pages = (len + kPage - 1) / kPage;
    const int per = (n_pages + n_splits - 1) / n_splits;
    const int lo = split * per, hi = min(n_pages, lo + per);
    const float C[4] = {fmt == 2 ? KeyCodebook<2>::C0 : KeyCodebook<1>::C0, fmt == 2 ? KeyCodebook<2>::C1 : KeyCodebook<1>::C1,
                        fmt == 2 ? KeyCodebook<2>::C2 : KeyCodebook<1>::C2, fmt == 2 ? KeyCodebook<2>::C3 : KeyCodebook<1>::C3};

    for (int g = 0; g < 8; ++g) {
        float x = g < G ? __bfloat162float(q[((size_t)b * hq + h * G + g) * D + tid]) : 0.f;
        qs[g * D + tid] = x;
        qr[g * D + tid] = ((sigma.w[tid >> 5] >> (tid & 31)) & 1u) ? -x : x;
    }
    __syncthreads();
    for (int hh = 1; hh < D; hh <<= 1) {
        float u[8];
        for (int g = 0; g < 8; ++g) {
            const float own = qr[g * D + tid], other = qr[g * D + (tid ^ hh)];
            u[g] = (tid & hh) ? other - own : own + other;
        }
        __syncthreads();
        for (int g = 0; g < 8; ++g) qr[g * D + tid] = u[g];
        __syncthreads();
    }
    const float rs = rsqrtf((float)D);
    for (int g = 0; g < 8; ++g) qr[g * D + tid] *= rs;
    __syncthreads();

    float O[8], m[8], l[8];
    for (int g = 0; g < 8; ++g) { O[g] = 0.f; m[g] = -CUDART_INF_F; l[g] = 0.f; }

    // `pg` counts 16-token tiles; the table has one entry per page of `tiles` tiles (tiles = 1: 16-token pages)
    for (int pg = lo; pg < hi; ++pg) {
        const int entry = pg / tiles, tile = pg - entry * tiles;
        const int tag = tags[(size_t)b * max_pages + entry], id = bt[(size_t)b * max_pages + entry];
        const int valid = min(kPage, len - pg * kPage);
        const bool is_tq3 = tag == MKV_TAG_STALE;
        const bool ok = is_tq3 ? (id >= 0 && id < tq3_pages && valid == kPage)
                               : (tag <= MKV_TAG_ANCHOR && id >= 0 && id < fp8_pages);
        if (!ok) {   // never fault: flag and treat the page as empty
            if (tid == 0) atomicOr(status, kStBounds);
            continue;
        }
        if (is_tq3) {
            // one tile of the page: key codes, value codes and g as in a 16-token record; the value scale/zero
            // of the page follow its last tile
            const uint8_t* page = tq3 + ((size_t)id * hkv + h) * tq3_page_bytes(D, tiles);
            const uint8_t* rec = page + (size_t)tile * tq3_tile_bytes(D);
            const int cb = tid >> 4, row = tid & 15;
            const __half* meta = reinterpret_cast<const __half*>(page + (size_t)tiles * tq3_tile_bytes(D));
            const int mi = (cb >> 1) * 64 + (row & 7) * 8 + 4 * (cb & 1) + (row >> 3);
            const float vsc = __half2float(meta[mi]), vzp = __half2float(meta[mi + 2]);
            for (int t = 0; t < kPage; ++t) {
                const int kc = tq3_key_code<D>(rec, t, tid, fmt);
                Ks[t * (D + 1) + tid] = (kc & 4) ? -C[kc & 3] : C[kc & 3];
                Vs[t * D + tid] = fmaf(vsc, (float)tq3_value_code<D>(rec, t, tid), vzp);
            }
            if (tid < kPage) gn[tid] = __half2float(reinterpret_cast<const __half*>(rec + 12 * D)[tid]);
        } else {
            const uint8_t* rec = fp8 + (((size_t)id * hkv + h) * tiles + tile) * fp8_record_bytes(D);
            for (int t = 0; t < kPage; ++t) {
                Ks[t * (D + 1) + tid] = e4m3_f32(rec[t * D + tid]) * k_scale;
                Vs[t * D + tid] = e4m3_f32(rec[16 * D + tid * kPage + t]) * v_scale;
            }
            if (tid < kPage) gn[tid] = 1.f;
        }
        __syncthreads();
        {   // 16 tokens x 8 heads dot products; D = 256 uses two threads per product
            const int pair = tid & 127, partn = tid >> 7, t = pair & 15, g = pair >> 4;
            const float* qx = (is_tq3 ? qr : qs) + g * D;
            constexpr int SPAN = D == 256 ? 128 : 128;
            float acc = 0.f;
            for (int c = partn * SPAN; c < partn * SPAN + SPAN; ++c) acc = fmaf(Ks[t * (D + 1) + c], qx[c], acc);
            red[partn * 128 + pair] = acc;
        }
        __syncthreads();
        if (tid < 128) {
            const int t = tid & 15;
            float s = red[tid];
            if (D == 256) s += red[128 + tid];
            s = s * scale * gn[t];
            sc[tid] = t < valid ? s : -CUDART_INF_F;     // sc[g*16 + t]
        }
        __syncthreads();
        for (int g = 0; g < G; ++g) {
            float mx = -CUDART_INF_F;
            for (int t = 0; t < kPage; ++t) mx = fmaxf(mx, sc[g * 16 + t]);
            const float mn = fmaxf(m[g], mx);
            if (mn == -CUDART_INF_F) continue;
            const float alpha = __expf(m[g] - mn);      // exp(-inf) = 0 on the first page
            float ls = 0.f, acc = 0.f;
            for (int t = 0; t < kPage; ++t) {
                const float pt = __expf(sc[g * 16 + t] - mn);
                ls += pt;
                acc = fmaf(pt, Vs[t * D + tid], acc);
            }
            l[g] = l[g] * alpha + ls;
            O[g] = O[g] * alpha + acc;
            m[g] = mn;
        }
        __syncthreads();
    }
    for (int g = 0; g < G; ++g) {
        float* dst = part + (((size_t)b * hq + h * G + g) * n_splits + split) * (D + 2);
        dst[tid] = O[g];
        if (tid == 0) { dst[D] = m[g]; dst[D + 1] = l[g]; }
    }
}

// Eq. (softmax-merge) over the splits of one (request, query head); O_j arrive unnormalised
// (l_j * normalised O_j).
template <int D>
__global__ void __launch_bounds__(D) merge_scalar_kernel(const float* __restrict__ part, int n_splits, int hq,
                                                          float* __restrict__ out, float* __restrict__ lse)
{
    const int head = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    const float* src = part + ((size_t)b * hq + head) * n_splits * (D + 2);
    float m = -CUDART_INF_F;
    for (int j = 0; j < n_splits; ++j) m = fmaxf(m, src[j * (D + 2) + D]);
    float l = 0.f, acc = 0.f;
    for (int j = 0; j < n_splits; ++j) {
        const float mj = src[j * (D + 2) + D], lj = src[j * (D + 2) + D + 1];
        if (lj > 0.f) {
            const float w = __expf(mj - m);
            l += w * lj;
            acc += w * src[j * (D + 2) + tid];
        }
    }
    out[((size_t)b * hq + head) * D + tid] = l > 0.f ? acc / l : 0.f;
    if (lse && tid == 0) lse[(size_t)b * hq + head] = l > 0.f ? m + logf(l) : -CUDART_INF_F;
}

template <int D>
static int32_t run_scalar(mkv_pool* p, const void* q, const int32_t* bt, const uint8_t* tags, const int32_t* lens,
                          int B, int max_pages, float scale, float* out, float* lse, void* ws, cudaStream_t s)
{
    const int S = scalar_splits(B, p->hkv);
    float* part = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + decode_ws_header_bytes(B, p->hkv));
    const size_t smem = sizeof(float) * (16 * D + kPage * (D + 1) + kPage * D + 256 + 128 + 16);
    static bool attr_done[2] = {false, false};
    if (!attr_done[D == 256]) {
        MKV_CUDA(cudaFuncSetAttribute(decode_scalar_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_done[D == 256] = true;
    }
    dim3 grid(S, p->hkv, B);
    decode_scalar_kernel<D><<<grid, D, smem, s>>>(p->fp8, p->tq3, p->cfg.fp8_pages, p->cfg.tq3_pages, p->hkv,
                                                  p->group, p->cfg.k_scale, p->cfg.v_scale, p->sigma,
                                                  (const __nv_bfloat16*)q, bt, tags, lens, max_pages, p->tiles, p->fmt, scale, S,
                                                  part, p->status_dev);
    MKV_CUDA(cudaGetLastError());
    merge_scalar_kernel<D><<<dim3(p->hq, B), D, 0, s>>>(part, S, p->hq, out, lse);
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
}

int32_t launch_decode_scalar(mkv_pool* p, const void* q, const int32_t* bt, const uint8_t* tags,
                             const int32_t* lens, int B, int max_pages, float scale, float* out, float* lse,
                             void* ws, size_t, cudaStream_t s)
{
    return p->d == 128 ? run_scalar<128>(p, q, bt, tags, lens, B, max_pages, scale, out, lse, ws, s)
                       : run_scalar<256>(p, q, bt, tags, lens, B, max_pages, scale, out, lse, ws, s);
}

}  // namespace mkv
