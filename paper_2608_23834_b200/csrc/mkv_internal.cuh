// Internal declarations of libmkv (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <utility>
#include <vector>

#include "mkv.h"

namespace mkv {

constexpr int kPage = 16;            // tokens per page
constexpr int kMaxGroup = 8;         // query heads per KV head handled by one MMA column block
constexpr int kStatusTail = 256;     // bytes reserved behind the FP8 records for the status word

// device status bits
constexpr uint32_t kStBounds = 1u, kStState = 2u, kStTimeout = 4u;

// TQ3 key codebook (8-level Lloyd-Max quantiser of N(0,1), levels rounded to fp16) and its
// decision thresholds (midpoints).  Section 3.1, "three-bit rotated scalar quantizer".
#define MKV_C0 0.2451171875f
#define MKV_C1 0.755859375f
#define MKV_C2 1.34375f
#define MKV_C3 2.15234375f
#define MKV_B0 0.50048828125f
#define MKV_B1 1.0498046875f
#define MKV_B2 1.748046875f

// Record format 2: the same quantiser with its levels on the nearest e4m3 numbers (0.25, 0.75, 1.375, 2.25), so
// that a reader feeds the codes to FP8 arithmetic exactly; thresholds are again the midpoints.
template <int FMT>
struct KeyCodebook {
    static constexpr float C0 = MKV_C0, C1 = MKV_C1, C2 = MKV_C2, C3 = MKV_C3;
    static constexpr float B0 = MKV_B0, B1 = MKV_B1, B2 = MKV_B2;
};
template <>
struct KeyCodebook<2> {
    static constexpr float C0 = 0.25f, C1 = 0.75f, C2 = 1.375f, C3 = 2.25f;
    static constexpr float B0 = 0.5f, B1 = 1.0625f, B2 = 1.8125f;
};

struct SigmaBits {
    uint32_t w[8];   // bit i set <=> rotation sign of dim i is -1
};

__host__ __device__ inline size_t fp8_record_bytes(int d) { return (size_t)32 * d; }
__host__ __device__ inline size_t tq3_record_bytes(int d) { return (size_t)16 * d + 32; }
// Pages of `tiles` 16-token tiles (Section 4.1 stores blocks of 1,792 / 832 tokens): an FP8 page is `tiles`
// consecutive 16-token records; a TQ3 page is `tiles` tile records (key codes, value codes, g: 12 d + 32
// bytes each) followed by ONE set of value scale/zero (4 d bytes) shared by all its tokens.  tiles = 1 gives
// the 16-token records above.
__host__ __device__ inline size_t tq3_tile_bytes(int d) { return (size_t)12 * d + 32; }
__host__ __device__ inline size_t fp8_page_bytes(int d, int tiles) { return (size_t)tiles * 32 * d; }
__host__ __device__ inline size_t tq3_page_bytes(int d, int tiles) { return (size_t)tiles * (12 * d + 32) + (size_t)4 * d; }
constexpr int kMaxTiles = 256;       // pages of at most 4,096 tokens

// ---- TQ3 record geometry -------------------------------------------------------------------
// The code sections are laid out for the m16n8k16 A-fragment: "lane" L = 4*g + tq owns rows
// g, g+8 and column slots 2tq, 2tq+1, 2tq+8, 2tq+9 of every 16x16 block.  A lane's 32-bit words
// are stored in 16-byte chunks (a trailing 8-byte chunk when two words remain).
__host__ __device__ inline int lane_words(int d) { return 3 * (d / 16) / 4; }
__host__ __device__ inline int lane_word_offset(int d, int lane, int w)
{
    int chunk = w >> 2, rem = lane_words(d) - 4 * chunk;
    return chunk * 512 + lane * (rem >= 4 ? 16 : 8) + (w & 3) * 4;
}

struct Device {
    int sm_count = 0;
    int max_smem_optin = 0;
};

}  // namespace mkv

struct mkv_pool {
    mkv_pool_config cfg;
    int d, hkv, hq, group;
    int tiles;                   // 16-token tiles per page (cfg.page_size / 16)
    int fmt;                     // TQ3 record format: 1 or 2 (cfg.tq3_format, 0 meaning 1)
    uint8_t* fp8;
    uint8_t* tq3;
    uint32_t* status_dev;
    mkv::SigmaBits sigma;
    int variant;
    unsigned long long wait_ns;  // wall-time limit of the decode scan's waits for a page copy
    int device;
    mkv::Device dev;
    std::mutex mu;
    std::vector<int32_t> free_list[2];
    std::vector<uint8_t> allocated[2];   // 0 free, 1 allocated, 2 retiring (source of a planned conversion)
};

struct mkv_seq {
    mkv_pool* pool;
    int32_t len;
    std::vector<int32_t> ids;
    std::vector<uint8_t> tags;
    std::vector<std::pair<int32_t, int32_t>> retiring;   // (format, id) of conversion sources awaiting mkv_seq_release
};

namespace mkv {
int32_t cuda_fail(cudaError_t e, const char* what);
#define MKV_CUDA(call)                                         \
    do {                                                       \
        cudaError_t e__ = (call);                              \
        if (e__ != cudaSuccess) return ::mkv::cuda_fail(e__, #call); \
    } while (0)

int32_t launch_append(mkv_pool* p, const void* k, const void* v, const int32_t* slots, int n, cudaStream_t s);
int32_t launch_demote(mkv_pool* p, const int32_t* src, const int32_t* dst, int n, int32_t* bt, uint8_t* tags,
                      const int64_t* entry, int64_t n_entries, cudaStream_t s);
int32_t launch_promote(mkv_pool* p, const int32_t* src, const int32_t* dst, int n, int32_t* bt, uint8_t* tags,
                       const int64_t* entry, int64_t n_entries, cudaStream_t s);
int32_t launch_set_anchor(mkv_pool* p, uint8_t* tags, int64_t entry, int flag, cudaStream_t s);
int32_t launch_decode_scalar(mkv_pool* p, const void* q, const int32_t* bt, const uint8_t* tags,
                             const int32_t* lens, int B, int max_pages, float scale, float* out, float* lse,
                             void* ws, size_t ws_bytes, cudaStream_t s);
int32_t launch_decode_tensor(mkv_pool* p, const void* q, const int32_t* bt, const uint8_t* tags,
                             const int32_t* lens, int B, int max_pages, float scale, float* out, float* lse,
                             void* ws, size_t ws_bytes, cudaStream_t s);
int32_t launch_decode_tensor_at(mkv_pool* p, const void* q, const int32_t* bt, const uint8_t* tags,
                                const int32_t* lens, int B, int max_pages, float scale, float* out, float* lse,
                                float* partials, uint32_t* tickets, int max_blocks, float* mass, cudaStream_t s);
int32_t launch_decode_tensor_layers(mkv_pool* const* pools, const void* const* q, const int32_t* const* bt,
                                    const uint8_t* const* tags, const int32_t* lens, int B, int max_pages, float scale,
                                    float* const* out, float* const* lse, void* const* ws, int n_layers, cudaStream_t s);
int32_t launch_append_layers(mkv_pool* const* pools, const void* const* k, const void* const* v, const int32_t* slots,
                             int n_tokens, int n_layers, cudaStream_t s);
int32_t launch_page_score(const float* mass, const int32_t* lens, int B, int hq, int max_pages, uint64_t head_mask,
                          float beta, float* score, int page_tokens, cudaStream_t s);
constexpr int kMaxCtas = 512;        // upper bound of the decode scan's persistent grid (sizes workspace and tickets)
int decode_tensor_partial_floats(int d);
void set_last_error(const char* msg);
size_t decode_ws_header_bytes(int B, int hkv);
size_t decode_ws_scalar_bytes(int B, int hkv, int group, int d);
size_t decode_ws_tensor_bytes(int B, int hkv, int group, int d);
int scalar_splits(int B, int hkv);
}  // namespace mkv
