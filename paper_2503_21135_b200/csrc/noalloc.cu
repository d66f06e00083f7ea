// Routing + permutation entry point for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at all: code running inside a CUDA-graph
// capture or under a memory pool that forbids new allocations, plugins that are handed a fixed
// set of buffers by their framework, and real-time loops that must not hit the allocator.  The
// regular forward takes its scratch from a caller-allocated workspace; this variant of the
// routing / permutation step keeps the scratch of the scan kernel (per-expert counts, the row of
// every (token, slot) pair, the token and expert of every sorted row) in a file-scope device array
// instead, so the caller passes only inputs and outputs.
#include "../../include/dynamo.h"
#include "common.cuh"

namespace dyn {
cudaError_t launch_route(const float* logits, int T, int E, int k, int renorm, int32_t* idx, float* w,
                         cudaStream_t st);
cudaError_t launch_scan(const WsDev& ws, int E, int Es, int k, cudaStream_t st);
}  // namespace dyn

namespace {

constexpr int NOALLOC_MAX_PAIRS = DYNAMO_NOALLOC_MAX_PAIRS;  // T * k
constexpr int NOALLOC_MAX_EXPERTS = 256;
// counts [256] | padded offsets [264] | pos [pairs] | row_token, row_expert [pairs + 8 * 256 padding rows]
constexpr size_t NOALLOC_ROWS = (size_t)NOALLOC_MAX_PAIRS + 8 * NOALLOC_MAX_EXPERTS;
constexpr size_t SCRATCH_INTS = 256 + 264 + (size_t)NOALLOC_MAX_PAIRS + 2 * NOALLOC_ROWS;

// Every GPU that loads the library holds this array (about 400 KiB) until the process exits.
static __device__ __align__(256) int32_t g_route_scratch[SCRATCH_INTS];

// In host code `g_route_scratch` is only a stand-in for the symbol, not a device address: the
// address each device gave the array is looked up once per device and cached here.
constexpr int MAX_DEVICES = 64;
int32_t* g_scratch_addr[MAX_DEVICES] = {nullptr};

cudaError_t scratch_for_current_device(int32_t** out) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        err = cudaGetSymbolAddress(&p, g_route_scratch);
        if (err != cudaSuccess) return err;
        g_scratch_addr[dev] = static_cast<int32_t*>(p);
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" dynamo_status dynamo_route_permute_static(const float* router_logits, int32_t T, int32_t n_experts,
                                                     int32_t top_k, int32_t renormalize, int32_t* topk_idx,
                                                     float* topk_w, int32_t* expert_offsets, int32_t* perm,
                                                     void* stream) {
    if (n_experts < 1 || n_experts > NOALLOC_MAX_EXPERTS || top_k < 1 || top_k > 8 || top_k > n_experts)
        return DYNAMO_ERR_SHAPE;
    if (T < 0 || (long long)T * top_k > NOALLOC_MAX_PAIRS) return DYNAMO_ERR_TOKENS;
    if (T == 0) return DYNAMO_OK;
    if (!router_logits || !topk_idx || !topk_w || !expert_offsets || !perm) return DYNAMO_ERR_NULL;
    int32_t* scratch = nullptr;
    if (scratch_for_current_device(&scratch) != cudaSuccess) return DYNAMO_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    dyn::WsDev ws = {};
    ws.counts = scratch;
    ws.off_pad = scratch + 256;
    ws.pos = scratch + 256 + 264;
    ws.row_token = ws.pos + NOALLOC_MAX_PAIRS;
    ws.row_expert = ws.row_token + NOALLOC_ROWS;
    ws.offsets = expert_offsets;
    ws.topk_idx = topk_idx;
    ws.topk_w = topk_w;
    ws.perm = perm;
    ws.T = T;
    ws.R = T * top_k;
    ws.ksplit = 1;
    if (dyn::launch_route(router_logits, T, n_experts, top_k, renormalize ? 1 : 0, topk_idx, topk_w, st) !=
        cudaSuccess)
        return DYNAMO_ERR_CUDA;
    // The scan kernel writes every scratch word it later reads, so nothing has to be cleared between calls.
    if (dyn::launch_scan(ws, n_experts, 0, top_k, st) != cudaSuccess) return DYNAMO_ERR_CUDA;
    return DYNAMO_OK;
}
