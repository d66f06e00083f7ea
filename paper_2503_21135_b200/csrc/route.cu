// Routing, permutation, activation gather and weighted combine kernels.
//
// route   : top-k of the router logits per token (ties -> lower expert index), softmax weights.
// scan    : expert histogram -> exclusive scan -> stable counting sort of the (token, slot) pairs
//           (token-ascending inside an expert), warp-ballot ranking: deterministic, no atomics order.
// gather  : expert-contiguous activation rows in fp16, significant columns zeroed for switchable
//           experts (they are served by the 8-bit path), per-64 sums, plus the gathered significant columns.
// combine : y[t] = sum_j w[t,j] * Y[pos(t,j)] + sum_shared Y[pos], fp32, fixed order.
#include "common.cuh"
#include "layout.cuh"

namespace dyn {

// One warp per token.  E <= 256: lane l holds logits l, l+32, ...
__global__ void __launch_bounds__(256) route_kernel(const float* __restrict__ logits, int T, int E, int k, int renorm,
                                                    int32_t* __restrict__ topk_idx, float* __restrict__ topk_w) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= T) return;
    const float* l = logits + (long long)warp * E;
    float v[8];
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int e = lane + 32 * i;
        v[i] = (e < E) ? l[e] : -INFINITY;
        mx = fmaxf(mx, v[i]);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float den = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i)
        if (lane + 32 * i < E) den += expf(v[i] - mx);
#pragma unroll
    for (int o = 16; o; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);

    float wsel[8];
    int isel[8];
    float wsum = 0.f;
    for (int j = 0; j < k; ++j) {
        // local best (value desc, index asc)
        float bv = -INFINITY;
        int bi = 0x7fffffff;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int e = lane + 32 * i;
            if (e < E && (v[i] > bv || (v[i] == bv && e < bi))) { bv = v[i]; bi = e; }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        // remove the winner from its owner's candidates (experts already taken are marked by index)
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (lane + 32 * i == bi) v[i] = -INFINITY;
        isel[j] = bi;
        wsel[j] = expf(bv - mx) / den;
        wsum += wsel[j];
    }
    if (lane == 0) {
        for (int j = 0; j < k; ++j) {
            topk_idx[(long long)warp * k + j] = isel[j];
            topk_w[(long long)warp * k + j] = renorm ? wsel[j] / wsum : wsel[j];
        }
    }
}

// Single CTA.  Warp w ranks the pairs of experts w, w + nwarps, ...  Pair order i = t*k + j is
// ascending in t, and a token holds an expert at most once, so rank-by-scan-order is the stable order.
__global__ void __launch_bounds__(1024) scan_kernel(WsDev ws, int E, int Es, int k) {
    __shared__ int s_count[MAX_EXPERTS + 1];
    __shared__ int s_off[MAX_EXPERTS + 1];
    const int T = ws.T, n_pairs = T * k;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int kk = k + Es;
    for (int e = warp; e < E; e += nwarps) {
        int c = 0;
        for (int base = 0; base < n_pairs; base += 32) {
            const int i = base + lane;
            const bool hit = (i < n_pairs) && (ws.topk_idx[i] == e);
            c += __popc(__ballot_sync(0xffffffffu, hit));
        }
        if (lane == 0) s_count[e] = c;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int acc = 0;
        for (int e = 0; e < E; ++e) { s_off[e] = acc; acc += s_count[e]; }
        s_off[E] = acc;  // = T*k
        for (int s = 0; s < Es; ++s) { s_count[E + s] = T; s_off[E + s + 1] = s_off[E + s] + T; }
    }
    __syncthreads();
    for (int e = threadIdx.x; e <= E + Es; e += blockDim.x) {
        ws.offsets[e] = s_off[e];
        if (e < E + Es) ws.counts[e] = s_count[e];
    }
    for (int e = warp; e < E; e += nwarps) {
        int run = s_off[e];
        for (int base = 0; base < n_pairs; base += 32) {
            const int i = base + lane;
            const bool hit = (i < n_pairs) && (ws.topk_idx[i] == e);
            const unsigned m = __ballot_sync(0xffffffffu, hit);
            if (hit) {
                const int r = run + __popc(m & ((1u << lane) - 1));
                const int t = i / k, j = i - t * k;
                ws.perm[r] = i;
                ws.pos[t * kk + j] = r;
                ws.row_token[r] = t;
                ws.row_expert[r] = e;
            }
            run += __popc(m);
        }
    }
    // shared experts: every token, natural order
    for (int i = threadIdx.x; i < Es * T; i += blockDim.x) {
        const int s = i / T, t = i - s * T;
        const int r = n_pairs + i;
        ws.pos[t * kk + k + s] = r;
        ws.row_token[r] = t;
        ws.row_expert[r] = E + s;
    }
}

// One CTA per sorted row; warp w converts chunks w, w+8, ...  The fp16 activations are stored
// multiplied by 2^x_scale_exp(bits of the row's expert, k) so that the FFN kernel can use packed codes
// in place; the per-64 sums are of the unscaled fp16 values.
__global__ void __launch_bounds__(256) gather_kernel(const LayerDev* __restrict__ L, WsDev ws,
                                                     const __nv_bfloat16* __restrict__ x) {
    const int row = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = ws.row_token[row], e = ws.row_expert[row];
    const int d = L->d;
    const int bits = L->ex[e].bits;
    const bool sw = L->ex[e].switchable != 0;
    const uint32_t* mask = sw ? (L->sigmask + (long long)e * (d / 32)) : nullptr;
    const __nv_bfloat16* xr = x + (long long)t * d;
    uint8_t* out = ws.xperm + (long long)row * (d / KC) * XROW;
    const float sc0 = __uint_as_float((uint32_t)(127 + x_scale_exp(bits, 4 * lane)) << 23);
    const float sc1 = __uint_as_float((uint32_t)(127 + x_scale_exp(bits, 4 * lane + 2)) << 23);
    for (int c = warp; c < d / KC; c += 8) {
        const int k0 = c * KC + lane * 4;
        const uint2 raw = *reinterpret_cast<const uint2*>(xr + k0);
        const __nv_bfloat162 p0 = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
        const __nv_bfloat162 p1 = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
        float v[4] = {__low2float(p0), __high2float(p0), __low2float(p1), __high2float(p1)};
        if (sw) {
            const uint32_t mw = mask[k0 >> 5] >> (k0 & 31);
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if ((mw >> i) & 1u) v[i] = 0.f;
        }
        float hv[4];
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            hv[i] = __half2float(__float2half_rn(v[i]));
            sum += hv[i];
        }
        // sum over the 16 lanes of each half chunk (64 k), fixed butterfly order
#pragma unroll
        for (int o = 8; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        const __half2 oa = __floats2half2_rn(hv[0] * sc0, hv[1] * sc0), ob = __floats2half2_rn(hv[2] * sc1, hv[3] * sc1);
        uint2 packed;
        packed.x = *reinterpret_cast<const uint32_t*>(&oa);
        packed.y = *reinterpret_cast<const uint32_t*>(&ob);
        *reinterpret_cast<uint2*>(out + (long long)c * XROW + lane * 8) = packed;
        if ((lane & 15) == 0)
            *reinterpret_cast<float*>(out + (long long)c * XROW + XROW_SUM_OFF + (lane >> 4) * 4) = sum;
    }
    // gathered significant columns (unscaled)
    const int S_pad = L->S_pad;
    const int cnt = sw ? L->sig_cnt[e] : 0;
    for (int j = threadIdx.x; j < S_pad; j += blockDim.x) {
        __half hv = __float2half_rn(0.f);
        if (j < cnt) hv = __float2half_rn(__bfloat162float(xr[L->sig_chan[e * S_pad + j]]));
        ws.xsig[(long long)row * S_pad + j] = hv;
    }
}

// grid (T, ceil(d / 1024)): each thread owns four output columns of one token.
__global__ void __launch_bounds__(256) combine_kernel(WsDev ws, int d, int k, int Es, void* __restrict__ y,
                                                      int y_f32, long long split_stride) {
    const int t = blockIdx.x;
    const int kk = k + Es;
    const int c = (blockIdx.y * blockDim.x + threadIdx.x) * 4;
    if (c >= d) return;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int j = 0; j < kk; ++j) {
        const int r = ws.pos[t * kk + j];
        const float w = (j < k) ? ws.topk_w[t * k + j] : 1.0f;
        float s[4] = {0.f, 0.f, 0.f, 0.f};
        for (int sp = 0; sp < ws.ksplit; ++sp) {
            const float4 v = *reinterpret_cast<const float4*>(ws.ypart + sp * split_stride + (long long)r * d + c);
            s[0] += v.x; s[1] += v.y; s[2] += v.z; s[3] += v.w;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = fmaf(w, s[i], acc[i]);
    }
    if (y_f32) {
        *reinterpret_cast<float4*>((float*)y + (long long)t * d + c) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    } else {
        __nv_bfloat162 a = __floats2bfloat162_rn(acc[0], acc[1]), b = __floats2bfloat162_rn(acc[2], acc[3]);
        uint2 o;
        o.x = *reinterpret_cast<uint32_t*>(&a);
        o.y = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint2*>((__nv_bfloat16*)y + (long long)t * d + c) = o;
    }
}

cudaError_t launch_route(const float* logits, int T, int E, int k, int renorm, int32_t* idx, float* w,
                         cudaStream_t st) {
    route_kernel<<<(T + 7) / 8, 256, 0, st>>>(logits, T, E, k, renorm, idx, w);
    return cudaGetLastError();
}
cudaError_t launch_scan(const WsDev& ws, int E, int Es, int k, cudaStream_t st) {
    const int warps = E < 32 ? (E < 1 ? 1 : E) : 32;
    scan_kernel<<<1, warps * 32, 0, st>>>(ws, E, Es, k);
    return cudaGetLastError();
}
cudaError_t launch_gather(const LayerDev* L, const WsDev& ws, const void* x, cudaStream_t st) {
    gather_kernel<<<ws.R, 256, 0, st>>>(L, ws, (const __nv_bfloat16*)x);
    return cudaGetLastError();
}
cudaError_t launch_combine(const WsDev& ws, int d, int k, int Es, void* y, int y_f32, long long split_stride,
                           cudaStream_t st) {
    combine_kernel<<<dim3((unsigned)ws.T, (unsigned)((d + 1023) / 1024)), 256, 0, st>>>(ws, d, k, Es, y, y_f32, split_stride);
    return cudaGetLastError();
}

}  // namespace dyn
