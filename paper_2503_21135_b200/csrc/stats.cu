// Runtime selection of the significant channels (Sections IV-B, V-A: the channels with the most prominent
// dynamics are the ones switched when the data changes; only cached channels can be served at high precision).
//
// stats  : while forwards run, per routed expert e and cached channel c the activation mass
//              A[e][c] += sum over the tokens routed to e in this forward of |x[t][c]|
//          is accumulated in fp32 in a FIXED order (the expert's rows are cut into slices, one CTA each: tokens
//          ascending inside a slice, slices ascending, one addition of the forward's sum to the running total),
//          so the numbers are reproducible bit for bit for a given slice count.
// select : per expert the S cached channels with the largest A (ties -> lower channel index) become the
//          significant set, in rank order; the index tables and the channel bitmask are rewritten on the
//          device exactly as a host-driven switch would write them.
#include "common.cuh"

namespace dyn {

// grid (E, n_slices), 256 threads: CTA (e, s) walks slice s of the expert's rows, thread j for cached channel j, and
// leaves its partial sums in `part` [E][n_slices][P_pad] (scratch: the down GEMM's output buffer, not yet in use at
// this point of a forward); the CTA that finishes last for an expert (a self-resetting counter per expert) adds the
// slices up in slice order and adds the result to the running total.
__global__ void __launch_bounds__(256) stats_kernel(const LayerDev* __restrict__ L, WsDev ws,
                                                    const __nv_bfloat16* __restrict__ x, float* __restrict__ stats,
                                                    float* __restrict__ part, int32_t* __restrict__ ctr) {
    __shared__ int s_last;
    pdl_prologue();
    const int e = blockIdx.x, s = blockIdx.y, nsl = gridDim.y;
    const int P = L->P, P_pad = L->P_pad, d = L->d;
    const int cnt = ws.counts[e], row0 = ws.off_pad[e];
    if (cnt == 0) return;  // every slice of the expert leaves: its counter stays at zero
    const int len = (cnt + nsl - 1) / nsl;
    const int r0 = min(cnt, s * len), r1 = min(cnt, r0 + len);
    const int32_t* ci = L->cache_idx + (long long)e * P;
    float* mine = part + ((long long)e * nsl + s) * P_pad;
    for (int j = threadIdx.x; j < P; j += blockDim.x) {
        const int ch = ci[j];
        float sum = 0.f;
#pragma unroll 4
        for (int r = r0; r < r1; ++r) {
            const int t = ws.row_token[row0 + r];
            sum += fabsf(__bfloat162float(x[(long long)t * d + ch]));
        }
        if (nsl == 1) stats[(long long)e * P_pad + j] += sum;   // a single slice: no second pass
        else mine[j] = sum;
    }
    if (nsl == 1) return;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(&ctr[e], 1) == nsl - 1) ? 1 : 0;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int j = threadIdx.x; j < P; j += blockDim.x) {
        float tot = 0.f;
        for (int q = 0; q < nsl; ++q) tot += __ldcg(part + ((long long)e * nsl + q) * P_pad + j);
        stats[(long long)e * P_pad + j] += tot;
    }
    if (threadIdx.x == 0) ctr[e] = 0;
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

// part: scratch of E * n_slices * P_pad floats; ctr: E zero-initialised counters (left at zero).
cudaError_t launch_stats(const LayerDev* L, const WsDev& ws, const void* x, float* stats, float* part, int32_t* ctr, int E,
                         int n_slices, cudaStream_t st) {
    return launch_pdl(stats_kernel, dim3((unsigned)E, (unsigned)n_slices), dim3(256), 0, st, L, ws,
                      (const __nv_bfloat16*)x, stats, part, ctr);
}

cudaError_t launch_select(const LayerDev* L, float* stats, int E, int P, int n_sel, int reset, int32_t* chosen,
                          cudaStream_t st) {
    select_kernel<<<(unsigned)E, 256, (size_t)P * sizeof(float), st>>>(L, stats, n_sel, reset, chosen);
    return cudaGetLastError();
}

}  // namespace dyn
