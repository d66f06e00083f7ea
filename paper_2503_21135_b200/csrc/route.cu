// Routing, permutation, activation gather and weighted combine kernels.
//
// route   : top-k of the router logits per token (ties -> lower expert index), softmax weights.
// scan    : expert histogram -> exclusive scan -> stable counting sort of the (token, slot) pairs
//           (token-ascending inside an expert), warp-ballot ranking: deterministic, no atomics order.
//           Also lays the experts' segments out in PHYSICAL rows (each segment starts at a multiple of 8).
// gather  : expert-contiguous activation rows in fp16, pre-scaled for in-place code use, significant
//           columns zeroed for switchable experts (they are served by the 8-bit path), per-group sums,
//           plus the gathered significant columns; written in the layout of the FFN path the row's
//           expert takes (streaming rows, or 8-row MMA operand tiles).
// combine : y[t] = sum_j w[t,j] * Y[pos(t,j)] + sum_shared Y[pos], fp32, fixed order.
#include "common.cuh"
#include "layout.cuh"

namespace dyn {

// Top-k of one token's logits held across a warp (lane l holds logits l, l+32, ...; E <= 256): k largest raw
// logits, descending, ties -> lower expert index; weights = softmax over all E restricted to the chosen,
// rescaled to sum 1 if `renorm`.
__device__ __forceinline__ void topk_softmax_store(float (&v)[8], int lane, int E, int k, int renorm, long long token,
                                                   int32_t* __restrict__ topk_idx, float* __restrict__ topk_w) {
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < 8; ++i) mx = fmaxf(mx, v[i]);
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
        // remove the winner from its owner's candidates
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (lane + 32 * i == bi) v[i] = -INFINITY;
        isel[j] = bi;
        wsel[j] = expf(bv - mx) / den;
        wsum += wsel[j];
    }
    if (lane == 0) {
        for (int j = 0; j < k; ++j) {
            topk_idx[token * k + j] = isel[j];
            topk_w[token * k + j] = renorm ? wsel[j] / wsum : wsel[j];
        }
    }
}

// One warp per token.
__global__ void __launch_bounds__(256) route_kernel(const float* __restrict__ logits, int T, int E, int k, int renorm,
                                                    int32_t* __restrict__ topk_idx, float* __restrict__ topk_w) {
    pdl_prologue();
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= T) return;
    const float* l = logits + (long long)warp * E;
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int e = lane + 32 * i;
        v[i] = (e < E) ? l[e] : -INFINITY;
    }
    topk_softmax_store(v, lane, E, k, renorm, warp, topk_idx, topk_w);
}

// Router GEMM fused with the top-k (Section II-A: the gate scores every expert, the K best are taken):
// logits[t][e] = sum_c x[t][c] * W_r[e][c] (+ bias[e]), bf16 inputs, fp32 accumulate.  One CTA of eight warps
// per token: warp w, lane l take the input indices 8*l + 256*(w + 8*i) ..+7; every warp reduces its partial
// sums over its lanes by a fixed butterfly, the eight partials are added in warp order, so the sum order
// (hence the fp32 result) is deterministic.  The products of two bf16 values are exact in fp32; only the
// additions round.  Warp 0 then selects the top-k exactly as route_kernel does.
__global__ void __launch_bounds__(256) route_gemm_kernel(const __nv_bfloat16* __restrict__ x,
                                                         const __nv_bfloat16* __restrict__ w_router,
                                                         const float* __restrict__ bias, int T, int d, int E, int k,
                                                         int renorm, float* __restrict__ logits_out,
                                                         int32_t* __restrict__ topk_idx, float* __restrict__ topk_w) {
    __shared__ float part[8][MAX_EXPERTS];
    pdl_prologue();
    const int token = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const __nv_bfloat16* xr = x + (long long)token * d;
    for (int e0 = 0; e0 < E; e0 += 8) {  // eight experts at a time
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.f;
        for (int c = 8 * lane + 256 * warp; c < d; c += 2048) {
            const uint4 xv = *reinterpret_cast<const uint4*>(xr + c);
            const __nv_bfloat162* xp = reinterpret_cast<const __nv_bfloat162*>(&xv);
            float xf[8];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                xf[2 * u] = __low2float(xp[u]);
                xf[2 * u + 1] = __high2float(xp[u]);
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (e0 + j < E) {
                    const uint4 wv = *reinterpret_cast<const uint4*>(w_router + (long long)(e0 + j) * d + c);
                    const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&wv);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        acc[j] = fmaf(xf[2 * u], __low2float(wp[u]), acc[j]);
                        acc[j] = fmaf(xf[2 * u + 1], __high2float(wp[u]), acc[j]);
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
            for (int o = 16; o; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
            if (lane == 0 && e0 + j < E) part[warp][e0 + j] = acc[j];
        }
    }
    __syncthreads();
    if (warp != 0) return;
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int e = lane + 32 * i;
        v[i] = -INFINITY;
        if (e < E) {
            float sum = part[0][e];
#pragma unroll
            for (int w = 1; w < 8; ++w) sum += part[w][e];
            v[i] = sum + (bias ? bias[e] : 0.f);
            if (logits_out) logits_out[(long long)token * E + e] = v[i];
        }
    }
    topk_softmax_store(v, lane, E, k, renorm, token, topk_idx, topk_w);
}

// Single CTA of 32 warps.  The pair array (pair i = t*k + j, ascending in t) is cut into 32 contiguous
// segments, one per warp.  Pass 1: each warp histograms its segment per expert (lanes holding the same
// expert find one another with match.any; the lowest lane of each group adds the group's size).
// An exclusive scan over segments turns the histograms into each segment's first rank within the
// expert; pass 2 walks the segment again and ranks each pair = segment base + pairs of that expert
// seen so far in the segment + position within the 32-pair batch.  Segments and lanes ascend in i and
// a token holds an expert at most once, so the rank is the stable order.
// offsets/perm are the logical (unpadded) permutation; pos/row_token/row_expert use physical rows.
__global__ void __launch_bounds__(1024) scan_kernel(WsDev ws, int E, int Es, int k) {
    __shared__ int s_hist[32][MAX_EXPERTS];
    __shared__ int s_count[MAX_EXPERTS + 1];
    __shared__ int s_off[MAX_EXPERTS + 1];
    __shared__ int s_pad[MAX_EXPERTS + 1];
    pdl_prologue();
    const int T = ws.T, n_pairs = T * k;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int kk = k + Es;
    // work-queue counters of this forward's streaming launches (callers that only route pass no status block)
    if (ws.status && threadIdx.x < 2) ws.status[4 + threadIdx.x] = 0;
    const int per_warp = ((n_pairs + 31) / 32 + nwarps - 1) / nwarps * 32;  // whole 32-pair batches per segment
    const int seg_lo = min(n_pairs, warp * per_warp), seg_hi = min(n_pairs, seg_lo + per_warp);
    const unsigned lt = (1u << lane) - 1;
    for (int e = lane; e < E; e += 32) s_hist[warp][e] = 0;
    __syncwarp();
    for (int base = seg_lo; base < seg_hi; base += 32) {
        const int i = base + lane;
        const bool valid = i < seg_hi;
        const int e = valid ? ws.topk_idx[i] : -1;
        const unsigned m = __match_any_sync(0xffffffffu, e);
        if (valid && (m & lt) == 0) s_hist[warp][e] += __popc(m);
        __syncwarp();
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E + Es; e += blockDim.x) {
        int acc = 0;
        if (e < E) {
            for (int w = 0; w < nwarps; ++w) {
                const int c = s_hist[w][e];
                s_hist[w][e] = acc;
                acc += c;
            }
        } else {
            acc = T;
        }
        s_count[e] = acc;
    }
    __syncthreads();
    if (warp == 0) {
        int run = 0, run_pad = 0;
        for (int e0 = 0; e0 < E + Es; e0 += 32) {
            const int e = e0 + lane;
            const int c = e < E + Es ? s_count[e] : 0;
            int v = c, vp = (c + 7) & ~7;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, v, d), up = __shfl_up_sync(0xffffffffu, vp, d);
                if (lane >= d) {
                    v += u;
                    vp += up;
                }
            }
            if (e < E + Es) {
                s_off[e] = run + v - c;
                s_pad[e] = run_pad + vp - ((c + 7) & ~7);
            }
            run += __shfl_sync(0xffffffffu, v, 31);
            run_pad += __shfl_sync(0xffffffffu, vp, 31);
        }
        if (lane == 0) {
            s_off[E + Es] = run;
            s_pad[E + Es] = run_pad;
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e <= E + Es; e += blockDim.x) {
        ws.offsets[e] = s_off[e];
        ws.off_pad[e] = s_pad[e];
        if (e < E + Es) ws.counts[e] = s_count[e];
    }
    for (int base = seg_lo; base < seg_hi; base += 32) {
        const int i = base + lane;
        const bool valid = i < seg_hi;
        const int e = valid ? ws.topk_idx[i] : -1;
        const unsigned m = __match_any_sync(0xffffffffu, e);
        const int start = valid ? s_hist[warp][e] : 0;
        __syncwarp();
        if (valid && (m & lt) == 0) s_hist[warp][e] = start + __popc(m);
        __syncwarp();
        if (valid) {
            const int r = start + __popc(m & lt);
            const int t = i / k, j = i - t * k;
            const int po = s_pad[e];
            ws.perm[s_off[e] + r] = i;
            ws.pos[t * kk + j] = po + r;
            ws.row_token[po + r] = t;
            ws.row_expert[po + r] = e;
        }
    }
    // padding rows of each routed expert's segment
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        const int c = s_count[e], po = s_pad[e];
        for (int r = c; r < ((c + 7) & ~7); ++r) {
            ws.row_token[po + r] = -1;
            ws.row_expert[po + r] = e;
        }
    }
    // shared experts: every token, natural order
    for (int s = 0; s < Es; ++s) {
        const int po = s_pad[E + s];
        const int padded = (T + 7) & ~7;
        for (int t = threadIdx.x; t < padded; t += blockDim.x) {
            if (t < T) ws.pos[t * kk + k + s] = po + t;
            ws.row_token[po + t] = t < T ? t : -1;
            ws.row_expert[po + t] = E + s;
        }
    }
}

// One CTA per physical row; warp w converts chunks w, w+8, ...  (Eight rows per CTA with one warp per row, so that
// the chain of dependent loads that finds a row's expert is paid once per eight rows, measured slower: +18 us on the
// 64-token step, nothing gained at 4096 tokens; staging a token's pair rows and weights in shared memory in the
// combine kernel measured no gain either.)  The fp16 activations are stored
// multiplied by 2^x_scale_exp(bits of the row's expert, k) so that the FFN kernels can use packed codes
// in place; the per-group sums are of the unscaled fp16 values.
__device__ __forceinline__ void gather_row(const LayerDev* __restrict__ L, const WsDev& ws,
                                           const __nv_bfloat16* __restrict__ x, int row, int t, int e, bool tc) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (t < 0 && !tc) return;  // padding rows matter only as zero rows of an MMA operand tile
    const int d = L->d;
    const int n_kc = d / KC;
    const int bits = L->ex[e].bits;
    const bool sw = L->ex[e].switchable != 0;
    const uint32_t* mask = sw ? (L->sigmask + (long long)e * (d / 32)) : nullptr;
    const __nv_bfloat16* xr = x + (long long)(t < 0 ? 0 : t) * d;
    const float sc0 = __uint_as_float((uint32_t)(127 + x_scale_exp(bits, 4 * lane)) << 23);
    const float sc1 = __uint_as_float((uint32_t)(127 + x_scale_exp(bits, 4 * lane + 2)) << 23);
    const int rg = row >> 3, rr = row & 7;
    bool clamped = false;
    for (int c = warp; c < n_kc; c += 8) {
        const int k0 = c * KC + lane * 4;
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (t >= 0) {
            const uint2 raw = *reinterpret_cast<const uint2*>(xr + k0);
            const __nv_bfloat162 p0 = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
            const __nv_bfloat162 p1 = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
            v[0] = __low2float(p0); v[1] = __high2float(p0); v[2] = __low2float(p1); v[3] = __high2float(p1);
#pragma unroll
            for (int i = 0; i < 4; ++i) v[i] = clamp_act(v[i], clamped);
            if (sw) {
                const uint32_t mw = mask[k0 >> 5] >> (k0 & 31);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if ((mw >> i) & 1u) v[i] = 0.f;
            }
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
        if (!tc) {
            uint8_t* out = ws.xperm + act_off(c, row, ws.Rcap);
            *reinterpret_cast<uint2*>(out + lane * 8) = packed;
            if ((lane & 15) == 0) *reinterpret_cast<float*>(out + XROW_SUM_OFF + (lane >> 4) * 4) = sum;
        } else {
            uint8_t* out = ws.xperm + act_off(c, 8 * rg, ws.Rcap);
            *reinterpret_cast<uint2*>(out + (lane >> 1) * 128 + rr * 16 + (lane & 1) * 8) = packed;
            // sums of the unscaled values per half chunk, beside the tile: [half 2][row 8] fp32
            if ((lane & 15) == 0) *reinterpret_cast<float*>(out + TC_TILE_BYTES + ((lane >> 4) * 8 + rr) * 4) = sum;
        }
    }
    if (clamped && ws.status) atomicOr(ws.status, STATUS_RANGE);
    // Activations of ALL cached channels of the row's expert, unscaled, zero where the channel is not
    // currently significant: the FFN kernels multiply them with the contiguous 8-bit-valued tiles of the
    // whole cache pool, so a switch only has to flip mask bits.
    if (!sw) return;
    const int P = L->P, P_pad = L->P_pad;
    const int32_t* ci = L->cache_idx + (long long)e * P;
    uint8_t* xp = reinterpret_cast<uint8_t*>(ws.xsig);
    for (int j = threadIdx.x; j < P_pad; j += blockDim.x) {
        const int pq = j >> 5, col = j & 31;
        if (!tc) {
            float v = 0.f;
            if (j < P) {
                const int ch = ci[j];
                if ((mask[ch >> 5] >> (ch & 31)) & 1u) v = clamp_act(__bfloat162float(xr[ch]), clamped);
            }
            *reinterpret_cast<__half*>(xp + xpool_off(pq, row, ws.Rcap) + col * 2) = __float2half_rn(v);
        } else {
            // operand position kp of a 16-column step holds pool column 16*step + sigma(kp): the A tile reaches
            // TMEM through an ldmatrix fragment whose k pairs (2t, 2t+1 | 2t+8, 2t+9) land on TMEM k 4t .. 4t+3.
            const int step = col >> 4, kp = col & 15;
            const int pj = pq * 32 + step * 16 + 2 * (kp >> 2) + (kp & 1) + ((kp & 2) ? 8 : 0);
            float v = 0.f;
            if (t >= 0 && pj < P) {
                const int ch = ci[pj];
                if ((mask[ch >> 5] >> (ch & 31)) & 1u) v = clamp_act(__bfloat162float(xr[ch]), clamped);
            }
            // 8-row operand tile of group pq: [k-octet 4][row 8][8 k] fp16 = 512 B
            *reinterpret_cast<__half*>(xp + xpool_off(pq, 8 * rg, ws.Rcap) + (col >> 3) * 128 + rr * 16 + (col & 7) * 2) =
                __float2half_rn(v);
        }
    }
}

__global__ void __launch_bounds__(256) gather_kernel(const LayerDev* __restrict__ L, WsDev ws,
                                                     const __nv_bfloat16* __restrict__ x) {
    pdl_prologue();
    const int row = blockIdx.x;
    if (row >= ws.off_pad[L->E + L->Es]) return;
    const int e = ws.row_expert[row];
    gather_row(L, ws, x, row, ws.row_token[row], e, ws.counts[e] > ws.tc_min);
}

// Small batches: routing, permutation and gather in ONE launch (three launches cost more than their work when the
// whole forward takes tens of microseconds).  One CTA per physical row; every CTA repeats the routing and the
// counting sort of all T * k pairs in shared memory (a few hundred pairs at most), then gathers its own row; CTA 0
// also writes the routing outputs and the row tables the later kernels read.  Same results as the three kernels.
constexpr int FRONT_MAX_PAIRS = 128;
constexpr int FRONT_MAX_TOKENS = 16;   // beyond this the three separate kernels are faster (measured at 32 and 64 tokens)
__global__ void __launch_bounds__(256) front_kernel(const LayerDev* __restrict__ L, WsDev ws,
                                                    const __nv_bfloat16* __restrict__ x,
                                                    const float* __restrict__ logits, int E, int Es, int k, int renorm) {
    __shared__ int s_idx[FRONT_MAX_PAIRS];
    __shared__ float s_w[FRONT_MAX_PAIRS];
    __shared__ int s_rank[FRONT_MAX_PAIRS];
    __shared__ int s_count[MAX_EXPERTS + 1], s_off[MAX_EXPERTS + 1], s_pad[MAX_EXPERTS + 1];
    __shared__ int s_row_e, s_row_t;
    pdl_prologue();
    const int T = ws.T, n_pairs = T * k, kk = k + Es;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int t = warp; t < T; t += 8) {
        const float* l = logits + (long long)t * E;
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int e = lane + 32 * i;
            v[i] = (e < E) ? l[e] : -INFINITY;
        }
        topk_softmax_store(v, lane, E, k, renorm, t, s_idx, s_w);
    }
    if (threadIdx.x == 0) { s_row_e = -1; s_row_t = -1; }
    __syncthreads();
    // counting sort: thread e walks the pairs in order (pair i = t*k + j ascends in t: the stable order)
    for (int e = threadIdx.x; e < E + Es; e += blockDim.x) {
        int c = 0;
        if (e < E) {
            for (int i = 0; i < n_pairs; ++i)
                if (s_idx[i] == e) s_rank[i] = c++;
        } else {
            c = T;
        }
        s_count[e] = c;
    }
    __syncthreads();
    if (warp == 0) {
        int run = 0, run_pad = 0;
        for (int e0 = 0; e0 < E + Es; e0 += 32) {
            const int e = e0 + lane;
            const int c = e < E + Es ? s_count[e] : 0;
            int v = c, vp = (c + 7) & ~7;
#pragma unroll
            for (int dd = 1; dd < 32; dd <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, v, dd), up = __shfl_up_sync(0xffffffffu, vp, dd);
                if (lane >= dd) {
                    v += u;
                    vp += up;
                }
            }
            if (e < E + Es) {
                s_off[e] = run + v - c;
                s_pad[e] = run_pad + vp - ((c + 7) & ~7);
            }
            run += __shfl_sync(0xffffffffu, v, 31);
            run_pad += __shfl_sync(0xffffffffu, vp, 31);
        }
        if (lane == 0) {
            s_off[E + Es] = run;
            s_pad[E + Es] = run_pad;
        }
    }
    __syncthreads();
    const int row = blockIdx.x;
    // whose row is this: the expert whose padded segment holds it, then the pair of that expert with this rank
    for (int e = threadIdx.x; e < E + Es; e += blockDim.x)
        if (row >= s_pad[e] && row < s_pad[e + 1]) s_row_e = e;
    __syncthreads();
    const int my_e = s_row_e;
    if (my_e >= 0) {
        const int r = row - s_pad[my_e];
        if (my_e < E) {
            for (int i = threadIdx.x; i < n_pairs; i += blockDim.x)
                if (s_idx[i] == my_e && s_rank[i] == r) s_row_t = i / k;
        } else if (threadIdx.x == 0 && r < T) {
            s_row_t = r;
        }
    }
    if (blockIdx.x == 0) {
        if (threadIdx.x < 2) ws.status[4 + threadIdx.x] = 0;   // work-queue counters of the two streaming launches
        // the outputs and tables of the route and scan kernels
        for (int i = threadIdx.x; i < n_pairs; i += blockDim.x) {
            const int e = s_idx[i], r = s_rank[i], t = i / k, j = i - t * k;
            ws.topk_idx[i] = e;
            ws.topk_w[i] = s_w[i];
            ws.perm[s_off[e] + r] = i;
            ws.pos[t * kk + j] = s_pad[e] + r;
            ws.row_token[s_pad[e] + r] = t;
            ws.row_expert[s_pad[e] + r] = e;
        }
        for (int e = threadIdx.x; e <= E + Es; e += blockDim.x) {
            ws.offsets[e] = s_off[e];
            ws.off_pad[e] = s_pad[e];
            if (e < E + Es) ws.counts[e] = s_count[e];
        }
        for (int e = threadIdx.x; e < E; e += blockDim.x) {
            const int c = s_count[e], po = s_pad[e];
            for (int r = c; r < ((c + 7) & ~7); ++r) {
                ws.row_token[po + r] = -1;
                ws.row_expert[po + r] = e;
            }
        }
        for (int sx = 0; sx < Es; ++sx) {
            const int po = s_pad[E + sx];
            const int padded = (T + 7) & ~7;
            for (int t = threadIdx.x; t < padded; t += blockDim.x) {
                if (t < T) ws.pos[t * kk + k + sx] = po + t;
                ws.row_token[po + t] = t < T ? t : -1;
                ws.row_expert[po + t] = E + sx;
            }
        }
    }
    __syncthreads();
    if (my_e < 0) return;
    gather_row(L, ws, x, row, s_row_t, my_e, s_count[my_e] > ws.tc_min);
}

// grid (T, ceil(d / 1024)): each thread owns four output columns of one token.
__global__ void __launch_bounds__(256) combine_kernel(WsDev ws, int d, int k, int Es, void* __restrict__ y,
                                                      int y_f32, long long split_stride) {
    pdl_prologue();
    if (*ws.status & STATUS_TIMEOUT) return;  // the FFN kernels started nothing: leave y alone
    const int t = blockIdx.x;
    const int kk = k + Es;
    const int c = (blockIdx.y * blockDim.x + threadIdx.x) * 4;
    if (c >= d) return;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int j = 0; j < kk; ++j) {
        const int r = ws.pos[t * kk + j];
        const float w = (j < k) ? ws.topk_w[t * k + j] : 1.0f;
        float s[4] = {0.f, 0.f, 0.f, 0.f};
        const int ns = (ws.counts[ws.row_expert[r]] > ws.tc_min) ? 1 : ws.ksplit;  // the tensor-core path does not split K
        for (int sp = 0; sp < ns; ++sp) {
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
    return launch_pdl(route_kernel, dim3((unsigned)((T + 7) / 8)), dim3(256), 0, st, logits, T, E, k, renorm, idx, w);
}
cudaError_t launch_route_gemm(const void* x, const void* w_router, const float* bias, int T, int d, int E, int k,
                              int renorm, float* logits_out, int32_t* idx, float* w, cudaStream_t st) {
    return launch_pdl(route_gemm_kernel, dim3((unsigned)T), dim3(256), 0, st, (const __nv_bfloat16*)x,
                      (const __nv_bfloat16*)w_router, bias, T, d, E, k, renorm, logits_out, idx, w);
}
cudaError_t launch_scan(const WsDev& ws, int E, int Es, int k, cudaStream_t st) {
    const int batches = (ws.T * k + 31) / 32;  // one warp per segment of whole 32-pair batches
    const int warps = batches < 8 ? 8 : (batches > 32 ? 32 : batches);  // >= 8: the per-expert loops want threads
    return launch_pdl(scan_kernel, dim3(1), dim3((unsigned)(warps * 32)), 0, st, ws, E, Es, k);
}
cudaError_t launch_gather(const LayerDev* L, const WsDev& ws, const void* x, cudaStream_t st) {
    return launch_pdl(gather_kernel, dim3((unsigned)ws.Rpad), dim3(256), 0, st, L, ws, (const __nv_bfloat16*)x);
}
bool front_fits(int T, int k) { return T <= FRONT_MAX_TOKENS && T * k <= FRONT_MAX_PAIRS; }
cudaError_t launch_front(const LayerDev* L, const WsDev& ws, const void* x, const float* logits, int E, int Es, int k,
                         int renorm, cudaStream_t st) {
    return launch_pdl(front_kernel, dim3((unsigned)ws.Rpad), dim3(256), 0, st, L, ws, (const __nv_bfloat16*)x, logits, E,
                      Es, k, renorm);
}
cudaError_t launch_combine(const WsDev& ws, int d, int k, int Es, void* y, int y_f32, long long split_stride,
                           cudaStream_t st) {
    return launch_pdl(combine_kernel, dim3((unsigned)ws.T, (unsigned)((d + 1023) / 1024)), dim3(256), 0, st, ws, d, k, Es,
                      y, y_f32, split_stride);
}

}  // namespace dyn
