// glance_topk_static: the per-offset top-k + log-softmax step with its scratch in a fixed device array.
//
// Some callers of this library are not allowed to allocate device memory at all: a serving process that has
// handed the whole GPU to its own arena at start-up (so a later cudaMalloc fails or is forbidden by policy),
// a plug-in running inside a host framework's callback where allocation calls are off limits, or a
// latency-critical loop that cannot tolerate the implicit device-wide synchronisation an allocation may
// cause.  The regular path asks such callers for a workspace sized by glance_workspace_bytes(); this
// entry point needs none: the two-stage top-k keeps its per-warp candidates and partial log-sum-exp
// terms in the file-scope array below, which every GPU that loads the library holds until the process exits.
#include <mutex>

#include "kernels.cuh"

namespace {

constexpr size_t kStaticScratchBytes = 1u << 20;          // 1 MiB: the stated maximum
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_topk_scratch[kStaticScratchBytes];

std::mutex g_mutex;
void *g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the array on the current device.  In host code `g_topk_scratch` is only a handle for
// the runtime, not a device address, so the address is looked up once per device and cached.
int32_t scratch_for_current_device(void **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GLANCE_E_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_topk_scratch) != cudaSuccess || !p) return GLANCE_E_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return GLANCE_OK;
}

}  // namespace

extern "C" int32_t glance_topk_static(const float *logits, int32_t batch, int32_t block_B, int32_t vocab, int32_t k,
                                      int32_t *topk_ids, float *topk_lp, void *cuda_stream) {
    if (!logits || !topk_ids || !topk_lp) return GLANCE_E_INVALID_ARG;
    if (batch < 1 || block_B < 2 || block_B > glance::kMaxBlock || vocab < 2 || k < 1 || k > glance::kMaxTopk || k > vocab)
        return GLANCE_E_INVALID_ARG;
    const size_t rows = (size_t)batch * (block_B - 1);
    const size_t warps = (size_t)glance::topk_warps(vocab);
    const size_t cand_bytes = (rows * warps * k * 8 + 255) / 256 * 256;
    const size_t ml_bytes = rows * warps * 2 * 4;
    // beyond the fixed array, or more rows than one launch dimension holds: refuse, launch nothing
    if (cand_bytes + ml_bytes > kStaticScratchBytes || rows > 65535) return GLANCE_E_CAPACITY;
    void *base = nullptr;
    const int32_t rc = scratch_for_current_device(&base);
    if (rc != GLANCE_OK) return rc;
    // every slot of both regions that stage 2 reads is written by stage 1 of the same call, so nothing
    // has to be cleared between calls even though the array keeps the previous call's contents
    auto *cand = reinterpret_cast<unsigned long long *>(base);
    auto *ml = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(base) + cand_bytes);
    (void)cudaGetLastError();      // an earlier, unrelated launch error is not this call's failure
    glance::launch_topk(logits, batch, block_B, vocab, k, topk_ids, topk_lp, cand, ml, (cudaStream_t)cuda_stream);
    return cudaPeekAtLastError() == cudaSuccess ? GLANCE_OK : GLANCE_E_CUDA;
}
