// Tree attention for callers that cannot allocate device memory.
//
// Some embedders of this library run inside a memory arena they do not control: a serving process
// that has handed every byte of the device to its own pool at start-up, a plug-in loaded after
// that point, or a latency-critical loop in which cudaMalloc (a device-wide synchronising call)
// is forbidden. llmcad_tree_attention() needs a context, and creating one allocates its work
// buffers. The variant below needs no context: the few kilobytes of scratch it uses (per-node
// depth, position, ancestor bit rows and a status word) live in a static device array that comes
// with the library image, so nothing is allocated at any time.
#include <cstdio>

#include "attention_tc.cuh"
#include "common.cuh"

namespace {

constexpr int kMaxNodes = LLMCAD_MAX_TREE;      // 128 tree nodes
// depth[128] | pos[128] | anc[128][4] | status: 128*4 + 128*4 + 128*16 + 4 bytes, rounded up
constexpr size_t kScratchBytes = 4096;

// One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void *g_scratch_ptr[kMaxDevices] = {};          // device address of the array on each device

thread_local char g_err[160] = "";

}  // namespace

extern "C" const char *llmcad_noalloc_last_error(void) { return g_err; }

extern "C" int llmcad_tree_attention_noalloc(const void *q, const void *k, const void *v, int32_t n_heads, int32_t kv_stride,
                                             int32_t prefix_len, const int32_t *parent_idx, int32_t n, void *o,
                                             int32_t *status_out, void *stream)
{
    using namespace llmcad;
    if (!q || !k || !v || !parent_idx || !o) { snprintf(g_err, sizeof(g_err), "null pointer"); return LLMCAD_ERR_INVALID_ARG; }
    if (n < 1 || prefix_len < 0 || n_heads < 1 || kv_stride < prefix_len + n) {
        snprintf(g_err, sizeof(g_err), "bad sizes: n=%d prefix_len=%d n_heads=%d kv_stride=%d", n, prefix_len, n_heads, kv_stride);
        return LLMCAD_ERR_INVALID_ARG;
    }
    if (n > kMaxNodes) {
        snprintf(g_err, sizeof(g_err), "n=%d exceeds the %d nodes the static scratch holds", n, kMaxNodes);
        return LLMCAD_ERR_UNSUPPORTED;
    }
    if (n_heads > 65535) { snprintf(g_err, sizeof(g_err), "n_heads=%d exceeds 65535", n_heads); return LLMCAD_ERR_UNSUPPORTED; }
    // the kernels move rows as 16-byte vectors and bulk copies: a misaligned buffer would fault on the device
    if (((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) |
          reinterpret_cast<uintptr_t>(o)) & 15) != 0) {
        snprintf(g_err, sizeof(g_err), "q, k, v and o must be 16-byte aligned");
        return LLMCAD_ERR_INVALID_ARG;
    }

    // Set-up, once per device, with that device current: in host code the array's name is only a
    // stand-in, the address the kernels need comes from the runtime.
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        snprintf(g_err, sizeof(g_err), "no usable current device");
        return LLMCAD_ERR_CUDA;
    }
    // (two host threads making their first call at once both look the address up and store the same value)
    if (__atomic_load_n(&g_scratch_ptr[dev], __ATOMIC_ACQUIRE) == nullptr) {
        void *ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || ptr == nullptr) {
            snprintf(g_err, sizeof(g_err), "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
            return LLMCAD_ERR_CUDA;
        }
        __atomic_store_n(&g_scratch_ptr[dev], ptr, __ATOMIC_RELEASE);
    }
    unsigned char *base = static_cast<unsigned char *>(__atomic_load_n(&g_scratch_ptr[dev], __ATOMIC_ACQUIRE));
    TreeBuffers tb;
    tb.depth = reinterpret_cast<int32_t *>(base);
    tb.pos = reinterpret_cast<int32_t *>(base + 512);
    tb.anc = reinterpret_cast<uint32_t *>(base + 1024);
    tb.rope_cs = nullptr;
    int32_t *status = reinterpret_cast<int32_t *>(base + 1024 + 2048);

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps what the previous call left: the status word must start at zero
    cudaError_t e = cudaMemsetAsync(status, 0, sizeof(int32_t), st);
    if (e == cudaSuccess) e = launch_tree_prep(parent_idx, nullptr, n, prefix_len, 0, 0, 0.f, tb, status, st);
    if (e == cudaSuccess) {
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess) {
            // neither kernel needs global scratch; same choice as the regular entry point
            if (attention_prefers_t5(n))
                e = launch_attention_t5(q, k, v, n_heads, 128, kv_stride, prefix_len, n, tb.anc, o, sms, status, st, nullptr);
            else
                e = launch_attention_tc(q, k, v, n_heads, 128, kv_stride, prefix_len, n, tb.anc, o, nullptr, nullptr, sms, status, st, nullptr);
        }
    }
    if (e == cudaSuccess && status_out != nullptr)
        e = cudaMemcpyAsync(status_out, status, sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
    if (e != cudaSuccess) {
        snprintf(g_err, sizeof(g_err), "CUDA: %s", cudaGetErrorString(e));
        return LLMCAD_ERR_CUDA;
    }
    return LLMCAD_OK;
}
