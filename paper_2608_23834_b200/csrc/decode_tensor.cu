#include "mkv_internal.cuh"
namespace mkv {
size_t decode_ws_tensor_bytes(int, int, int, int) { return 0; }
int32_t launch_decode_tensor(mkv_pool*, const void*, const int32_t*, const uint8_t*, const int32_t*, int, int, float,
                             float*, float*, void*, size_t, cudaStream_t) { return MKV_E_INVALID; }
}
