// mkv_decode_attention_static: decode attention for callers that may not allocate device memory.
//
// Some users of this library cannot hand it a workspace: an inference server that gives its whole
// device memory budget to the KV pool when it starts and forbids cudaMalloc afterwards, a plug-in that
// runs inside somebody else's memory manager, a process whose allocator is locked down once serving
// begins.  For them the split partials (m, l, O) of the scan live in a fixed array that is part of
// the library image instead of a caller buffer.  The price is a fixed size and one shared copy:
// every GPU that loads the library carries the array until the process exits, and every call on a
// device uses the same array.
#include <mutex>

#include "mkv_internal.cuh"

namespace {

constexpr int kStaticMaxBlocks = MKV_STATIC_MAX_BLOCKS;
constexpr size_t kStaticBytes = MKV_STATIC_SCRATCH_BYTES;
constexpr size_t kPartialBytes = (size_t)2 * kStaticMaxBlocks * (8 * 256 + 16) * sizeof(float);   // d = 256
static_assert(kStaticBytes >= kPartialBytes + kStaticMaxBlocks * sizeof(uint32_t), "partials plus one ticket word per block");

// The scratch itself.  In host code this name is only a handle for the runtime, not an address a
// kernel could use; the device address is asked for once per device (below) and handed to the kernels.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {nullptr};

}  // namespace

extern "C" int32_t mkv_decode_attention_static(mkv_pool* pool, const void* q, const int32_t* bt, const uint8_t* tags,
                                               const int32_t* lens, int32_t B, int32_t max_pages, float scale,
                                               float* out, float* lse, void* stream)
{
    if (!pool || !pool->fp8 || B < 0 || max_pages < 0) return MKV_E_INVALID;
    if (B == 0) return MKV_OK;
    if (!q || !bt || !tags || !lens || !out) return MKV_E_INVALID;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out)) % 16) return MKV_E_INVALID;
    if (!(scale == scale)) return MKV_E_INVALID;
    if (B > MKV_STATIC_MAX_BATCH) {
        mkv::set_last_error("mkv_decode_attention_static: batch larger than MKV_STATIC_MAX_BATCH");
        return MKV_E_INVALID;
    }
    int dev = -1;
    MKV_CUDA(cudaGetDevice(&dev));
    if (dev != pool->device || dev < 0 || dev >= kMaxDevices) {
        mkv::set_last_error("mkv_decode_attention_static: the pool's device must be the current device");
        return MKV_E_INVALID;
    }
    if (pool->variant != MKV_DECODE_TENSOR) {
        // the fixed array is sized for the partials of the tensor-core scan; the other kernels keep theirs elsewhere
        mkv::set_last_error("mkv_decode_attention_static: runs the tensor-core kernel only; set the pool's decode variant back to MKV_DECODE_TENSOR");
        return MKV_E_INVALID;
    }
    void* scratch = nullptr;
    {
        // first call on this device: resolve the device address of the array (no allocation happens)
        std::lock_guard<std::mutex> lk(g_mu);
        if (!g_scratch_addr[dev]) {
            void* ptr = nullptr;
            MKV_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
            g_scratch_addr[dev] = ptr;
        }
        scratch = g_scratch_addr[dev];
    }
    // Partial slots are written before they are read.  The ticket words behind them start at zero
    // (the array is zero-initialised when the module is loaded) and every call leaves them at zero.
    uint32_t* tickets = reinterpret_cast<uint32_t*>(static_cast<unsigned char*>(scratch) + kPartialBytes);
    // A refusal keeps the reason the launch code recorded (a table wider than 65,535 tiles per row, more
    // blocks than MKV_STATIC_MAX_BLOCKS partial slots, a device index out of range): mkv_last_cuda_error().
    return mkv::launch_decode_tensor_at(pool, q, bt, tags, lens, B, max_pages, scale, out, lse,
                                        static_cast<float*>(scratch), tickets, kStaticMaxBlocks, nullptr,
                                        (cudaStream_t)stream);
}
