// gkv_decode_attn_static: one decode-attention step that needs no buffer beyond its inputs and
// outputs. The per-sequence length words, the completion and work counters and the status word that
// the context-based call keeps in a caller-allocated workspace live here in a fixed array inside the
// library's own device image. (The partial results of units split over the keys need no global
// scratch: they meet in the shared memory of a thread-block cluster.)
//
// It exists for callers that cannot obtain device memory at the point of the call: code running
// after an application has handed its whole memory budget to a pool it does not control (a plug-in
// inside an inference server), or latency-critical loops where cudaMalloc is forbidden because it
// synchronises the device and can fail late. Such a caller still owns q, k_new, v_new, the cache and
// out; it just has no way to produce a workspace.
//
// The array costs kStaticScratchBytes of device memory on every GPU that loads the library, until
// the process exits. All calls share it: two calls that overlap on the GPU (different streams, or
// different host threads without ordering) race on it and give wrong results.
#include <math.h>

#include <mutex>

#include "gkv_common.cuh"
#include "gkv_internal.h"

namespace {

using namespace gkv;

constexpr int kStaticMaxSeq = 1024;            // batch
constexpr size_t kOffStatus = 0;                                   // int32[64]: status word, work counters
constexpr size_t kOffLen = 256;                                    // int32[kStaticMaxSeq]
constexpr size_t kOffSeqDone = kOffLen + 4 * kStaticMaxSeq;        // int32[kStaticMaxSeq]
constexpr size_t kStaticScratchBytes = kOffSeqDone + 4 * kStaticMaxSeq;   // 8.25 KiB

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

__global__ void gkv_static_fill_len(int32_t* len, int n, int32_t value) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) len[i] = value;
}

// Device address of the array on the current device, resolved once per device.
constexpr int kMaxDevices = 64;
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_mu;
unsigned char* g_addr[kMaxDevices] = {};
int g_sm_count[kMaxDevices] = {};
bool g_ready[kMaxDevices] = {};
EncodeFn g_encode = nullptr;     // the driver's tensor-map encoder, looked up once per process

// Set-up on the first call per device (with that device current): the array's device address, the SM count, the
// decode kernel's shared-memory attribute, and -- once per process -- the tensor-map encoder. Later calls only read.
gkv_status scratch_for_current_device(unsigned char** out, int* sm_count) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GKV_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_ready[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
            (void)cudaGetLastError();
            return GKV_ERR_CUDA;
        }
        if (decode_kernel_setup() != cudaSuccess ||
            cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return GKV_ERR_CUDA;
        }
        if (!g_encode) {
            void* sym = nullptr;
            cudaDriverEntryPointQueryResult q;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
                q != cudaDriverEntryPointSuccess || !sym) {
                (void)cudaGetLastError();
                return GKV_ERR_CUDA;
            }
            g_encode = reinterpret_cast<EncodeFn>(sym);
        }
        g_addr[dev] = static_cast<unsigned char*>(p);
        g_ready[dev] = true;
    }
    *out = g_addr[dev];
    *sm_count = g_sm_count[dev];
    return GKV_OK;
}

// [rows][128] bf16 view in boxes of box_rows rows x 64 elements with the 128-byte swizzle the decode kernel expects.
bool encode_rows(CUtensorMap* map, void* base, uint64_t rows, uint32_t box_rows) {
    const cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)kRowBytes};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr,
                                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

extern "C" gkv_status gkv_decode_attn_static(const void* q, const void* k_new, const void* v_new, void* k_cache,
                                             void* v_cache, void* out, int32_t batch, int32_t n_q_heads,
                                             int32_t n_kv_heads, int32_t capacity, int32_t len, void* stream) {
    if (!q || !k_new || !v_new || !k_cache || !v_cache || !out) return GKV_ERR_INVALID_ARG;
    if (batch <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || capacity <= 0 || len < 0) return GKV_ERR_INVALID_ARG;
    if (n_q_heads % n_kv_heads != 0) return GKV_ERR_INVALID_ARG;
    if (n_q_heads / n_kv_heads > kMaxGroup || capacity > 4096) return GKV_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(k_cache) | reinterpret_cast<uintptr_t>(v_cache) | reinterpret_cast<uintptr_t>(q) |
         reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) | reinterpret_cast<uintptr_t>(out)) % 16 != 0)
        return GKV_ERR_INVALID_ARG;
    if (len >= capacity) return GKV_ERR_CAPACITY;
    const long units = (long)batch * n_kv_heads;
    if (batch > kStaticMaxSeq) return GKV_ERR_SCRATCH_LIMIT;

    unsigned char* scratch = nullptr;
    int sm = 0;
    gkv_status st = scratch_for_current_device(&scratch, &sm);
    if (st != GKV_OK) return st;

    DecodeLaunch p;
    p.n_layers = 1; p.batch = batch; p.h_kv = n_kv_heads; p.C = capacity;
    p.accum = 0;
    p.sm_count = sm;
    decode_plan(&p, 0);
    DecodeMaps maps;
    const uint64_t rows = (uint64_t)units * capacity;
    if (rows >= (1ull << 31)) return GKV_ERR_UNSUPPORTED;   // TMA row coordinate is a signed 32-bit integer
    if (!encode_rows(&maps.k64, k_cache, rows, kTileKeys) || !encode_rows(&maps.v64, v_cache, rows, kTileKeys) ||
        !encode_rows(&maps.k16, k_cache, rows, 16) || !encode_rows(&maps.v16, v_cache, rows, 16))
        return GKV_ERR_CUDA;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call left: status word and counters must start at zero,
    // and every sequence's length word is set to this call's `len`.
    if (cudaMemsetAsync(scratch, 0, kStaticScratchBytes, s) != cudaSuccess) return GKV_ERR_CUDA;
    int32_t* d_len = reinterpret_cast<int32_t*>(scratch + kOffLen);
    gkv_static_fill_len<<<(batch + 255) / 256, 256, 0, s>>>(d_len, batch, len);
    if (cudaGetLastError() != cudaSuccess) return GKV_ERR_CUDA;

    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_new = static_cast<const __nv_bfloat16*>(k_new);
    p.v_new = static_cast<const __nv_bfloat16*>(v_new);
    p.out = static_cast<__nv_bfloat16*>(out);
    p.k_cache = static_cast<__nv_bfloat16*>(k_cache);
    p.v_cache = static_cast<__nv_bfloat16*>(v_cache);
    p.sacc = nullptr;
    p.len = d_len;
    p.seq_done = reinterpret_cast<int32_t*>(scratch + kOffSeqDone);
    p.status = reinterpret_cast<int32_t*>(scratch + kOffStatus);
    p.work_next = p.status + 32;
    p.layer0 = 0; p.n_layers = 1; p.batch = batch; p.h_q = n_q_heads; p.h_kv = n_kv_heads;
    p.g = n_q_heads / n_kv_heads; p.C = capacity;
    p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)kHeadDim));
    if (launch_decode(p, maps, s) != cudaSuccess) {
        (void)cudaGetLastError();
        return GKV_ERR_CUDA;
    }
    return GKV_OK;
}
