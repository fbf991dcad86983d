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
template <int D>
__global__ void __launch_bounds__(D / 2) append_kernel(uint8_t* __restrict__ fp8, int fp8_pages, int hkv,
                                                        float inv_k_scale, float inv_v_scale,
                                                        const __nv_bfloat162* __restrict__ k,
                                                        const __nv_bfloat162* __restrict__ v,
                                                        const int32_t* __restrict__ slots,
                                                        uint32_t* __restrict__ status)
{
    const int tok = blockIdx.x, h = blockIdx.y, i = threadIdx.x * 2;
    const int sm = slots[tok];
    if (sm < 0) return;
    const int page = sm >> 4, slot = sm & 15;
    if (page >= fp8_pages) {
        if (threadIdx.x == 0) atomicOr(status, kStBounds);
        return;
    }
    uint8_t* rec = fp8 + ((size_t)page * hkv + h) * fp8_record_bytes(D);
    const size_t src = ((size_t)tok * hkv + h) * (D / 2) + threadIdx.x;
    float2 kf = __bfloat1622float2(k[src]);
    float2 vf = __bfloat1622float2(v[src]);
    kf.x = __fmul_rn(kf.x, inv_k_scale);
    kf.y = __fmul_rn(kf.y, inv_k_scale);
    vf.x = __fmul_rn(vf.x, inv_v_scale);
    vf.y = __fmul_rn(vf.y, inv_v_scale);
    // round to nearest even, saturate to +-448
    __nv_fp8x2_storage_t kq = __nv_cvt_float2_to_fp8x2(kf, __NV_SATFINITE, __NV_E4M3);
    __nv_fp8x2_storage_t vq = __nv_cvt_float2_to_fp8x2(vf, __NV_SATFINITE, __NV_E4M3);
    *reinterpret_cast<uint16_t*>(rec + slot * D + i) = kq;             // K: token-major
    rec[16 * D + i * kPage + slot] = (uint8_t)(vq & 0xFF);             // V: channel-major
    rec[16 * D + (i + 1) * kPage + slot] = (uint8_t)(vq >> 8);
}

int32_t launch_append(mkv_pool* p, const void* k, const void* v, const int32_t* slots, int n, cudaStream_t s)
{
    dim3 grid(n, p->hkv);
    const float ik = 1.0f / p->cfg.k_scale, iv = 1.0f / p->cfg.v_scale;
    if (p->d == 128)
        append_kernel<128><<<grid, 64, 0, s>>>(p->fp8, p->cfg.fp8_pages, p->hkv, ik, iv,
                                               (const __nv_bfloat162*)k, (const __nv_bfloat162*)v, slots,
                                               p->status_dev);
    else
        append_kernel<256><<<grid, 128, 0, s>>>(p->fp8, p->cfg.fp8_pages, p->hkv, ik, iv,
                                                (const __nv_bfloat162*)k, (const __nv_bfloat162*)v, slots,
                                                p->status_dev);
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
}

// ------------------------------------------------------------------------------------------ demote
// One block per page; loops over the KV heads.  Warps encode key vectors (one token each), threads
// encode value channels, then all threads assemble the packed words from the codes in shared memory.
template <int D>
__global__ void __launch_bounds__(256) demote_kernel(const uint8_t* __restrict__ fp8, uint8_t* __restrict__ tq3,
                                                      int fp8_pages, int tq3_pages, int hkv, float k_scale,
                                                      float v_scale, SigmaBits sigma,
                                                      const int32_t* __restrict__ src_ids,
                                                      const int32_t* __restrict__ dst_ids, int32_t* block_table,
                                                      uint8_t* tier_tag, const int64_t* entry_index,
                                                      uint32_t* __restrict__ status)
{
    constexpr int EPL = D / 32;          // key elements per lane
    constexpr int LW = 3 * (D / 16) / 4; // packed words per lane and section
    __shared__ uint8_t kcode[kPage][D];
    __shared__ uint8_t vcode[kPage][D];
    __shared__ uint16_t g_s[kPage];
    __shared__ uint16_t sc_s[D], zp_s[D];

    const int page = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int src = src_ids[page], dst = dst_ids[page];
    if (src < 0 || src >= fp8_pages || dst < 0 || dst >= tq3_pages) {
        if (tid == 0) atomicOr(status, kStBounds);
        return;
    }
    const float C[4] = {MKV_C0, MKV_C1, MKV_C2, MKV_C3};

    for (int h = 0; h < hkv; ++h) {
        const uint8_t* rec8 = fp8 + ((size_t)src * hkv + h) * fp8_record_bytes(D);
        uint8_t* rec3 = tq3 + ((size_t)dst * hkv + h) * tq3_record_bytes(D);

        // ---- keys: warp w encodes tokens w and w + 8 ------------------------------------------
        for (int tok = warp; tok < kPage; tok += 8) {
            float x[EPL], a[EPL];
            const uint8_t* row = rec8 + tok * D + lane * EPL;
#pragma unroll
            for (int r = 0; r < EPL; ++r) {
                const int i = lane * EPL + r;
                x[r] = __fmul_rn(e4m3_to_f32(row[r]), k_scale);
                a[r] = ((sigma.w[i >> 5] >> (i & 31)) & 1u) ? -x[r] : x[r];
            }
            // Walsh-Hadamard butterflies, strides ascending: inside the lane, then across lanes
#pragma unroll
            for (int hh = 1; hh < EPL; hh <<= 1)
#pragma unroll
                for (int r = 0; r < EPL; ++r)
                    if ((r & hh) == 0) {
                        const float u = a[r], w = a[r + hh];
                        a[r] = __fadd_rn(u, w);
                        a[r + hh] = __fsub_rn(u, w);
                    }
#pragma unroll
            for (int m = 1; m < 32; m <<= 1)
#pragma unroll
                for (int r = 0; r < EPL; ++r) {
                    const float o = __shfl_xor_sync(0xffffffffu, a[r], m);
                    a[r] = (lane & m) ? __fsub_rn(o, a[r]) : __fadd_rn(a[r], o);
                }
            // |x|^2: pairwise tree in index order (every element of the butterfly ends equal)
            float e[EPL];
#pragma unroll
            for (int r = 0; r < EPL; ++r) e[r] = __fmul_rn(x[r], x[r]);
#pragma unroll
            for (int hh = 1; hh < EPL; hh <<= 1)
#pragma unroll
                for (int r = 0; r < EPL; r += 2 * hh) e[r] = __fadd_rn(e[r], e[r + hh]);
            float n2 = e[0];
#pragma unroll
            for (int m = 1; m < 32; m <<= 1) n2 = __fadd_rn(n2, __shfl_xor_sync(0xffffffffu, n2, m));
            const float nx = __fsqrt_rn(n2);
            const float t1 = __fmul_rn(MKV_B0, nx), t2 = __fmul_rn(MKV_B1, nx), t3 = __fmul_rn(MKV_B2, nx);
            float f[EPL];
#pragma unroll
            for (int r = 0; r < EPL; ++r) {
                const float w = fabsf(a[r]);
                const int mag = (w > t1) + (w > t2) + (w > t3);
                const int sgn = a[r] < 0.0f ? 1 : 0;
                kcode[tok][lane * EPL + r] = (uint8_t)(mag | (sgn << 2));
                f[r] = __fmul_rn(C[mag], C[mag]);
            }
#pragma unroll
            for (int hh = 1; hh < EPL; hh <<= 1)
#pragma unroll
                for (int r = 0; r < EPL; r += 2 * hh) f[r] = __fadd_rn(f[r], f[r + hh]);
            float nc2 = f[0];
#pragma unroll
            for (int m = 1; m < 32; m <<= 1) nc2 = __fadd_rn(nc2, __shfl_xor_sync(0xffffffffu, nc2, m));
            const float nc = __fsqrt_rn(nc2);
            if (lane == 0) g_s[tok] = (nx == 0.0f) ? (uint16_t)0 : f32_to_f16_sat_bits(__fdiv_rn(nx, nc));
        }

        // ---- values: one thread per channel, 16 tokens of the page ------------------------------
        for (int c = tid; c < D; c += 256) {
            const uint4 raw = *reinterpret_cast<const uint4*>(rec8 + 16 * D + c * kPage);
            const uint8_t* bytes = reinterpret_cast<const uint8_t*>(&raw);
            float val[kPage];
#pragma unroll
            for (int t = 0; t < kPage; ++t) val[t] = __fmul_rn(e4m3_to_f32(bytes[t]), v_scale);
            float mn = val[0], mx = val[0];
#pragma unroll
            for (int t = 1; t < kPage; ++t) {
                if (val[t] < mn) mn = val[t];
                if (val[t] > mx) mx = val[t];
            }
            const uint16_t sc = f32_to_f16_sat_bits(__fdiv_rn(__fsub_rn(mx, mn), 7.0f));
            const uint16_t zp = f32_to_f16_sat_bits(mn);
            const float scf = __half2float(__ushort_as_half(sc)), zpf = __half2float(__ushort_as_half(zp));
            sc_s[c] = sc;
            zp_s[c] = zp;
#pragma unroll
            for (int t = 0; t < kPage; ++t) {
                int q = 0;
                if (scf != 0.0f) {
                    float r = rintf(__fdiv_rn(__fsub_rn(val[t], zpf), scf));   // half to even
                    r = r < 0.0f ? 0.0f : r;
                    r = r > 7.0f ? 7.0f : r;
                    q = (int)r;
                }
                vcode[t][c] = (uint8_t)q;
            }
        }
        __syncthreads();

        // ---- pack: every thread assembles whole 32-bit words of the two code sections ----------
        for (int idx = tid; idx < 2 * 32 * LW; idx += 256) {
            const int section = idx / (32 * LW), L = (idx / LW) & 31, w = idx % LW;
            const int g = L >> 2, tq = L & 3, j = w / 3, kind = w % 3;
            uint32_t word = 0;
            if (section == 0) {
                // key codes: nibble n = 2r + half holds row g + 8(r&1), slot 2tq + 8(r>>1) + half
#pragma unroll
                for (int n = 0; n < 8; ++n) {
                    const int r = n >> 1, half = n & 1;
                    const int t = g + 8 * (r & 1), s = 2 * tq + 8 * (r >> 1) + half;
                    if (kind < 2) {   // A: block 4j (+ signs of block 4j+2); B: block 4j+1 (+ signs of 4j+3)
                        const uint32_t own = kcode[t][16 * (4 * j + kind) + s];
                        const uint32_t other = kcode[t][16 * (4 * j + kind + 2) + s];
                        word |= (own | ((other >> 2) << 3)) << (4 * n);
                    } else {          // C: magnitudes of blocks 4j+2 (low pair) and 4j+3 (high pair)
                        const uint32_t lo = kcode[t][16 * (4 * j + 2) + s] & 3u;
                        const uint32_t hi = kcode[t][16 * (4 * j + 3) + s] & 3u;
                        word |= (lo | (hi << 2)) << (4 * n);
                    }
                }
            } else {
                // value codes: four 24-bit streams (group, half) per triple, spread over 3 words
                uint32_t S[2][2];
#pragma unroll
                for (int grp = 0; grp < 2; ++grp)
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t st = 0;
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const int cb = 4 * j + 2 * grp + (k >> 2), r = k & 3;
                            const int row = g + 8 * (r & 1), t = 2 * tq + 8 * (r >> 1) + half;
                            st |= (uint32_t)vcode[t][16 * cb + row] << (3 * k);
                        }
                        S[grp][half] = st;
                    }
                auto byte = [](uint32_t st, int b) { return (st >> (8 * b)) & 0xFFu; };
                if (kind == 0)
                    word = byte(S[0][0], 0) | byte(S[0][0], 1) << 8 | byte(S[0][1], 0) << 16 | byte(S[0][1], 1) << 24;
                else if (kind == 1)
                    word = byte(S[0][0], 2) | byte(S[1][0], 0) << 8 | byte(S[0][1], 2) << 16 | byte(S[1][1], 0) << 24;
                else
                    word = byte(S[1][0], 1) | byte(S[1][0], 2) << 8 | byte(S[1][1], 1) << 16 | byte(S[1][1], 2) << 24;
            }
            *reinterpret_cast<uint32_t*>(rec3 + section * 6 * D + lane_word_offset(D, L, w)) = word;
        }
        if (tid < kPage) *reinterpret_cast<uint16_t*>(rec3 + 12 * D + 2 * tid) = g_s[tid];
        for (int c = tid; c < D; c += 256) {
            const int cb = c >> 4, row = c & 15;
            const int hi = (cb >> 1) * 64 + (row & 7) * 8 + 4 * (cb & 1) + (row >> 3);
            uint16_t* meta = reinterpret_cast<uint16_t*>(rec3 + 12 * D + 32);
            meta[hi] = sc_s[c];
            meta[hi + 2] = zp_s[c];
        }
        __syncthreads();
    }

    // copy-before-publish: the record is complete and visible before its id and tag appear
    __threadfence();
    __syncthreads();
    if (tid == 0 && entry_index != nullptr) {
        const int64_t e = entry_index[page];
        if (e >= 0) {
            block_table[e] = dst;
            __threadfence();
            tier_tag[e] = (uint8_t)MKV_TAG_STALE;
        }
    }
}

int32_t launch_demote(mkv_pool* p, const int32_t* src, const int32_t* dst, int n, int32_t* bt, uint8_t* tags,
                      const int64_t* entry, cudaStream_t s)
{
    if (p->d == 128)
        demote_kernel<128><<<n, 256, 0, s>>>(p->fp8, p->tq3, p->cfg.fp8_pages, p->cfg.tq3_pages, p->hkv,
                                             p->cfg.k_scale, p->cfg.v_scale, p->sigma, src, dst, bt, tags, entry,
                                             p->status_dev);
    else
        demote_kernel<256><<<n, 256, 0, s>>>(p->fp8, p->tq3, p->cfg.fp8_pages, p->cfg.tq3_pages, p->hkv,
                                             p->cfg.k_scale, p->cfg.v_scale, p->sigma, src, dst, bt, tags, entry,
                                             p->status_dev);
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
}

// ------------------------------------------------------------------------------------------ promote
// Promote (Algorithm 1 step 3): reconstruct a Stale page into a newly allocated FP8 page, then publish
// it as Anchor.  One block per page, loops over the KV heads.  Warps rebuild key vectors (signed
// levels, shuffle Walsh-Hadamard, norm correction, sign), threads rebuild value channels; the fp32
// operation order is fixed so that the written bytes are reproducible.
template <int D>
__device__ __forceinline__ uint32_t tq3_lane_word(const uint8_t* section, int lane, int w)
{
    return *reinterpret_cast<const uint32_t*>(section + lane_word_offset(D, lane, w));
}

template <int D>
__device__ int tq3_key_code_at(const uint8_t* rec, int t, int i)
{
    const int kb = i >> 4, s = i & 15;
    const int lane = 4 * (t & 7) + ((s & 7) >> 1), r = (t >> 3) + 2 * (s >> 3), n = 2 * r + (s & 1), j = kb >> 2;
    const uint32_t A = tq3_lane_word<D>(rec, lane, 3 * j), Bw = tq3_lane_word<D>(rec, lane, 3 * j + 1),
                   Cw = tq3_lane_word<D>(rec, lane, 3 * j + 2);
    switch (kb & 3) {
    case 0: return (A >> (4 * n)) & 7;
    case 1: return (Bw >> (4 * n)) & 7;
    case 2: return ((Cw >> (4 * n)) & 3) | (((A >> (4 * n + 3)) & 1) << 2);
    default: return ((Cw >> (4 * n + 2)) & 3) | (((Bw >> (4 * n + 3)) & 1) << 2);
    }
}

template <int D>
__device__ int tq3_value_code_at(const uint8_t* rec, int t, int c)
{
    const int cb = c >> 4, row = c & 15;
    const int lane = 4 * (row & 7) + ((t & 7) >> 1), r = (row >> 3) + 2 * (t >> 3), half = t & 1;
    const int j = cb >> 2, grp = (cb & 3) >> 1, k = 4 * (cb & 1) + r;
    const uint8_t* sec = rec + 6 * D;
    const uint32_t W0 = tq3_lane_word<D>(sec, lane, 3 * j), W1 = tq3_lane_word<D>(sec, lane, 3 * j + 1),
                   W2 = tq3_lane_word<D>(sec, lane, 3 * j + 2);
    auto by = [](uint32_t w, int b) { return (w >> (8 * b)) & 0xFFu; };
    uint32_t st;
    if (grp == 0)
        st = half == 0 ? (by(W0, 0) | by(W0, 1) << 8 | by(W1, 0) << 16) : (by(W0, 2) | by(W0, 3) << 8 | by(W1, 2) << 16);
    else
        st = half == 0 ? (by(W1, 1) | by(W2, 0) << 8 | by(W2, 1) << 16) : (by(W1, 3) | by(W2, 2) << 8 | by(W2, 3) << 16);
    return (st >> (3 * k)) & 7;
}

template <int D>
__global__ void __launch_bounds__(256) promote_kernel(const uint8_t* __restrict__ tq3, uint8_t* __restrict__ fp8,
                                                       int tq3_pages, int fp8_pages, int hkv, float inv_k_scale,
                                                       float inv_v_scale, float rs, SigmaBits sigma,
                                                       const int32_t* __restrict__ src_ids,
                                                       const int32_t* __restrict__ dst_ids, int32_t* block_table,
                                                       uint8_t* tier_tag, const int64_t* entry_index,
                                                       uint32_t* __restrict__ status)
{
    constexpr int EPL = D / 32;
    const int page = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int src = src_ids[page], dst = dst_ids[page];
    if (src < 0 || src >= tq3_pages || dst < 0 || dst >= fp8_pages) {
        if (tid == 0) atomicOr(status, kStBounds);
        return;
    }
    const float C[4] = {MKV_C0, MKV_C1, MKV_C2, MKV_C3};
    for (int h = 0; h < hkv; ++h) {
        const uint8_t* rec3 = tq3 + ((size_t)src * hkv + h) * tq3_record_bytes(D);
        uint8_t* rec8 = fp8 + ((size_t)dst * hkv + h) * fp8_record_bytes(D);
        // ---- keys: warp w rebuilds tokens w and w + 8
        for (int tok = warp; tok < kPage; tok += 8) {
            float y[EPL];
#pragma unroll
            for (int r = 0; r < EPL; ++r) {
                const int kc = tq3_key_code_at<D>(rec3, tok, lane * EPL + r);
                y[r] = (kc & 4) ? -C[kc & 3] : C[kc & 3];
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
            for (int m = 1; m < 32; m <<= 1)
#pragma unroll
                for (int r = 0; r < EPL; ++r) {
                    const float o = __shfl_xor_sync(0xffffffffu, y[r], m);
                    y[r] = (lane & m) ? __fsub_rn(o, y[r]) : __fadd_rn(y[r], o);
                }
            const float g = __half2float(reinterpret_cast<const __half*>(rec3 + 12 * D)[tok]);
            const float gr = __fmul_rn(g, rs);
#pragma unroll
            for (int r = 0; r < EPL; ++r) {
                const int i = lane * EPL + r;
                float k = __fmul_rn(gr, y[r]);
                if ((sigma.w[i >> 5] >> (i & 31)) & 1u) k = -k;
                rec8[tok * D + i] = (uint8_t)__nv_cvt_float_to_fp8(__fmul_rn(k, inv_k_scale), __NV_SATFINITE, __NV_E4M3);
            }
        }
        // ---- values: one thread per channel
        for (int c = tid; c < D; c += 256) {
            const int cb = c >> 4, row = c & 15;
            const __half* meta = reinterpret_cast<const __half*>(rec3 + 12 * D + 32);
            const int mi = (cb >> 1) * 64 + (row & 7) * 8 + 4 * (cb & 1) + (row >> 3);
            const float sc = __half2float(meta[mi]), zp = __half2float(meta[mi + 2]);
            uint32_t out[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int t = 0; t < kPage; ++t) {
                const float v = __fadd_rn(__fmul_rn(sc, (float)tq3_value_code_at<D>(rec3, t, c)), zp);
                const uint32_t b = (uint32_t)__nv_cvt_float_to_fp8(__fmul_rn(v, inv_v_scale), __NV_SATFINITE, __NV_E4M3);
                out[t >> 2] |= b << (8 * (t & 3));
            }
            *reinterpret_cast<uint4*>(rec8 + 16 * D + c * kPage) = make_uint4(out[0], out[1], out[2], out[3]);
        }
    }
    // copy-before-publish
    __threadfence();
    __syncthreads();
    if (tid == 0 && entry_index != nullptr) {
        const int64_t e = entry_index[page];
        if (e >= 0) {
            block_table[e] = dst;
            __threadfence();
            tier_tag[e] = (uint8_t)MKV_TAG_ANCHOR;
        }
    }
}

int32_t launch_promote(mkv_pool* p, const int32_t* src, const int32_t* dst, int n, int32_t* bt, uint8_t* tags,
                       const int64_t* entry, cudaStream_t s)
{
    const float ik = 1.0f / p->cfg.k_scale, iv = 1.0f / p->cfg.v_scale;
    const float rs = (float)(1.0 / sqrt((double)p->d));
    if (p->d == 128)
        promote_kernel<128><<<n, 256, 0, s>>>(p->tq3, p->fp8, p->cfg.tq3_pages, p->cfg.fp8_pages, p->hkv, ik, iv, rs,
                                              p->sigma, src, dst, bt, tags, entry, p->status_dev);
    else
        promote_kernel<256><<<n, 256, 0, s>>>(p->tq3, p->fp8, p->cfg.tq3_pages, p->cfg.fp8_pages, p->hkv, ik, iv, rs,
                                              p->sigma, src, dst, bt, tags, entry, p->status_dev);
    MKV_CUDA(cudaGetLastError());
    return MKV_OK;
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
