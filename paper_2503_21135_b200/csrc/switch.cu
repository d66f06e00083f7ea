// Runtime channel switch: installs the significant-channel tables of every expert of every layer
// of a switch event in one launch.  Only index tables and the per-expert channel bitmask are
// rewritten; packed base codes, base params and the cached 8-bit tiles are not touched.
#include "common.cuh"

namespace dyn {

// grid (E, n_layers).  staging: per layer [E][S_pad] channel per slot, [E][S_pad] pool position per
// slot, [E] counts (host-validated: in range, unique, members of the expert's cache).
__global__ void __launch_bounds__(128) switch_kernel(const SwitchLayers layers, const int32_t* __restrict__ staging,
                                                     int per_layer) {
    const int e = blockIdx.x, l = blockIdx.y;
    const LayerDev* L = layers.layer[l];
    const int S_pad = L->S_pad, E = L->E;
    const int32_t* chan = staging + (long long)l * per_layer + e * S_pad;
    const int32_t* pool = staging + (long long)l * per_layer + (E + e) * S_pad;
    const int cnt = staging[(long long)l * per_layer + 2 * E * S_pad + e];
    uint32_t* mask = L->sigmask + (long long)e * (L->d / 32);
    for (int i = threadIdx.x; i < L->d / 32; i += blockDim.x) mask[i] = 0u;
    __syncthreads();
    for (int j = threadIdx.x; j < S_pad; j += blockDim.x) {
        const int c = chan[j];
        L->sig_chan[e * S_pad + j] = c;
        L->sig_pool[e * S_pad + j] = pool[j];
        if (j < cnt) atomicOr(&mask[c >> 5], 1u << (c & 31));
    }
    if (threadIdx.x == 0) L->sig_cnt[e] = cnt;
}

cudaError_t launch_switch(const SwitchLayers& layers, int n_layers, int E, const int32_t* staging, int per_layer_ints,
                          cudaStream_t st) {
    dim3 grid((unsigned)E, (unsigned)n_layers);
    switch_kernel<<<grid, 128, 0, st>>>(layers, staging, per_layer_ints);
    return cudaGetLastError();
}

}  // namespace dyn
