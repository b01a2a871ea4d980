// Greedy verify/accept from logits for callers that must not allocate device memory.
//
// The ordinary entry point (dflash_verify_accept) takes its scratch - the per-segment winners of
// the row-wise argmax - from a workspace the caller allocated. Some callers cannot
// do that: a serving engine that has already handed every free byte of the GPU to its KV-cache
// pool, a latency-critical thread for which cudaMalloc's device-wide synchronisation is off limits,
// or code that is recording a stream into a CUDA graph. For them the same kernels run here on a
// fixed scratch array that is part of the library image: every GPU that loads the library carries
// it (about 1.1 MB) until the process exits, and nothing is allocated or freed at run time.
//
// Consequences the caller has to know:
//   * the array is shared by every call on the device and keeps whatever the previous call left in
//     it. Nothing in it has to start at zero: each call overwrites every entry it later reads.
//   * two calls that overlap on the GPU (different streams, no ordering between them) race on it.
//   * sizes above DFLASH_STATIC_MAX_ROWS rows are refused with DFLASH_ERR_UNSUPPORTED.
//   * the first call on each device looks up the array's device address (a host-side query, no
//     allocation); make that first call outside of any stream capture.
#include "dflash_internal.h"

#include <mutex>

namespace {

constexpr int kMaxRows = DFLASH_STATIC_MAX_ROWS;    // batch * (gamma + 1)
constexpr int kSegPerRow = 64;                      // upper bound of row_argmax_segments()
constexpr int kMaxDevices = 64;

struct StaticScratch {
    float4 seg[kMaxRows * kSegPerRow];   // per-(row, segment) winners of the argmax scan
};
// Device memory owned by the library image. In host code this name is only a handle for the
// runtime's symbol queries - never a pointer a kernel may be given.
static __device__ __align__(256) StaticScratch g_static_scratch;

std::mutex g_mu;
StaticScratch* g_dev_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device (resolved once per device).
int resolve(StaticScratch** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DFLASH_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_dev_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return DFLASH_ERR_CUDA;
        g_dev_ptr[dev] = static_cast<StaticScratch*>(p);
    }
    *out = g_dev_ptr[dev];
    return DFLASH_OK;
}

}  // namespace

extern "C" int32_t dflash_verify_accept_static(dflash_handle* h, const dflash_verify_args* a, void* stream) {
    using namespace dflash;
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (a->mode != DFLASH_VERIFY_LOGITS) return DFLASH_ERR_INVALID_ARG;      // ids mode needs no scratch at all
    if (a->batch < 0 || a->gamma < 1 || a->gamma > 64 || a->draft_stride < a->gamma) return DFLASH_ERR_INVALID_ARG;
    if (a->batch == 0) return DFLASH_OK;
    if (!a->logits || a->vocab < 2 || !a->draft_ids || !a->ctx_len || !a->accept_len || !a->out_tokens || !a->bonus ||
        !a->new_ctx_len)
        return DFLASH_ERR_INVALID_ARG;
    if (a->logits_dtype != DFLASH_F32 && a->logits_dtype != DFLASH_BF16) return DFLASH_ERR_UNSUPPORTED;
    const int64_t stride = a->logits_row_stride ? a->logits_row_stride : a->vocab;
    if (stride < a->vocab) return DFLASH_ERR_INVALID_ARG;
    const int64_t rows = (int64_t)a->batch * (a->gamma + 1);
    if (rows > kMaxRows) return DFLASH_ERR_UNSUPPORTED;       // beyond the fixed scratch: use dflash_verify_accept
    StaticScratch* s = nullptr;
    const int rc = resolve(&s);
    if (rc != DFLASH_OK) return rc;
    Launch L{h, (cudaStream_t)stream, a->dev_status, nullptr};
    return launch_verify_logits(L, *a, stride, s->seg);
}
