// Runtime selection of the significant channels (Sections IV-B, V-A: the channels with the most prominent
// dynamics are the ones switched when the data changes; only cached channels can be served at high precision).
//
// stats  : while forwards run, per routed expert e and cached channel c the activation mass
//              A[e][c] += sum over the tokens routed to e in this forward of |x[t][c]|
//          is accumulated in fp32 in a FIXED order (tokens ascending inside a forward, one addition of the
//          forward's sum to the running total), so the numbers are reproducible bit for bit.
// select : per expert the S cached channels with the largest A (ties -> lower channel index) become the
//          significant set, in rank order; the index tables and the channel bitmask are rewritten on the
//          device exactly as a host-driven switch would write them.
#include "common.cuh"

namespace dyn {

// grid (E), 256 threads: thread j walks the expert's rows for cached channel j.
__global__ void __launch_bounds__(256) stats_kernel(const LayerDev* __restrict__ L, WsDev ws,
                                                    const __nv_bfloat16* __restrict__ x, float* __restrict__ stats) {
    pdl_prologue();
    const int e = blockIdx.x;
    const int P = L->P, P_pad = L->P_pad, d = L->d;
    const int cnt = ws.counts[e], row0 = ws.off_pad[e];
    if (cnt == 0) return;
    const int32_t* ci = L->cache_idx + (long long)e * P;
    for (int j = threadIdx.x; j < P; j += blockDim.x) {
        const int ch = ci[j];
        float sum = 0.f;
        for (int r = 0; r < cnt; ++r) {
            const int t = ws.row_token[row0 + r];
            sum += fabsf(__bfloat162float(x[(long long)t * d + ch]));
        }
        stats[(long long)e * P_pad + j] += sum;
    }
}

// grid (E), 256 threads.  rank(j) = number of cached channels that beat j (larger A, or equal A and lower channel
// index); the channels of rank < n_sel fill the slots in rank order.  chosen: [E][S_pad] for the host mirror.
__global__ void __launch_bounds__(256) select_kernel(const LayerDev* __restrict__ L, float* __restrict__ stats, int n_sel,
                                                     int reset, int32_t* __restrict__ chosen) {
    extern __shared__ float sA[];  // [P]
    const int e = blockIdx.x;
    const int P = L->P, P_pad = L->P_pad, S_pad = L->S_pad, d = L->d;
    const int32_t* ci = L->cache_idx + (long long)e * P;
    const bool sw = L->ex[e].switchable != 0;
    const int cnt = sw ? min(n_sel, P) : 0;
    for (int j = threadIdx.x; j < P; j += blockDim.x) sA[j] = stats[(long long)e * P_pad + j];
    uint32_t* mask = L->sigmask + (long long)e * (d / 32);
    for (int i = threadIdx.x; i < d / 32; i += blockDim.x) mask[i] = 0u;
    for (int j = threadIdx.x; j < S_pad; j += blockDim.x) {
        L->sig_chan[e * S_pad + j] = -1;
        L->sig_pool[e * S_pad + j] = P;
        chosen[e * S_pad + j] = -1;
    }
    __syncthreads();
    for (int j = threadIdx.x; j < P; j += blockDim.x) {
        const float a = sA[j];
        int rank = 0;
        for (int i = 0; i < P; ++i) rank += (sA[i] > a || (sA[i] == a && i < j)) ? 1 : 0;  // cache_idx ascends with i
        if (rank < cnt) {
            const int c = ci[j];
            L->sig_chan[e * S_pad + rank] = c;
            L->sig_pool[e * S_pad + rank] = j;
            chosen[e * S_pad + rank] = c;
            atomicOr(&mask[c >> 5], 1u << (c & 31));
        }
        if (reset) stats[(long long)e * P_pad + j] = 0.f;
    }
    if (threadIdx.x == 0) L->sig_cnt[e] = cnt;
}

cudaError_t launch_stats(const LayerDev* L, const WsDev& ws, const void* x, float* stats, int E, cudaStream_t st) {
    return launch_pdl(stats_kernel, dim3((unsigned)E), dim3(256), 0, st, L, ws, (const __nv_bfloat16*)x, stats);
}

cudaError_t launch_select(const LayerDev* L, float* stats, int E, int P, int n_sel, int reset, int32_t* chosen,
                          cudaStream_t st) {
    select_kernel<<<(unsigned)E, 256, (size_t)P * sizeof(float), st>>>(L, stats, n_sel, reset, chosen);
    return cudaGetLastError();
}

}  // namespace dyn
