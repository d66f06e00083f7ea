// Significant channels on the d_ff side (Section IV-B applied to the second projection: the input channels of
// W_down are the hidden units).  A significant hidden unit c of expert e takes column c of the expert's uniform
// 8-bit quantization of W_down (same groups of G hidden units, same quantizer as pack).
//
// The down GEMM itself is untouched: it multiplies the fp16 h by the base-precision weights.  What a significant
// column adds is    y[row][n] += h[row][c] * (W8[n][c] - Wbase[n][c]),    and the difference is laid out at pack
// time as fp16 per (cached channel, output row), so a forward with S2 significant channels per expert costs one
// small kernel of rows x d x S2 multiply-adds between the down GEMM and the combine, and a switch is a table write.
//
// pack   : 8-bit parameters and the extrema of every (row, group) of W_down; for every cached channel its 8-bit code,
//          its bf16 original (the channel cache) and the fp16 difference to the base value.
// retarget: another target precision for an expert's cached channels (Section IV-B: requantized to the precision
//          the new data calls for): parameters from the stored extrema, codes and differences from the channel cache.
// requant: the same for the channels of a newly installed set only (switch mode "requantize from the cache").
// fix    : the correction above, reading h from the activation buffer in the layout the expert's path wrote it in.
// export : logical 8-bit codes and parameters for parity checks.
#include "common.cuh"
#include "layout.cuh"
#include "quant.cuh"

namespace dyn {

// One thread per output row n of W_down (d rows of f hidden units).
__global__ void pack_down_hi_kernel(const __nv_bfloat16* __restrict__ w_down, int d, int f, int G, int P2,
                                    const int32_t* __restrict__ cache_idx, int base_bits, DownExpertDev ex) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= d) return;
    const __nv_bfloat16* row = w_down + (long long)n * f;
    const int ng = f / G;
    int pi = 0;
    for (int g = 0; g < ng; ++g) {
        double lo = bf16_to_double(row[g * G]), hi = lo;
        for (int i = 1; i < G; ++i) {
            const double v = bf16_to_double(row[g * G + i]);
            lo = v < lo ? v : lo;
            hi = v > hi ? v : hi;
        }
        __half s_h, m_h;
        double s8, m8;
        group_params(lo, hi, HI_BITS, s_h, m_h, s8, m8);
        __half2 pr = __halves2half2(s_h, m_h);
        ex.s8m8[(long long)n * ng + g] = *reinterpret_cast<uint32_t*>(&pr);
        ex.gminmax[(long long)n * ng + g] = (uint32_t)__bfloat16_as_ushort(__double2bfloat16(lo)) |
                                            ((uint32_t)__bfloat16_as_ushort(__double2bfloat16(hi)) << 16);
        if (pi < P2 && cache_idx[pi] < (g + 1) * G) {
            double sb, mb;
            group_params(lo, hi, base_bits, s_h, m_h, sb, mb);
            while (pi < P2 && cache_idx[pi] < (g + 1) * G) {
                const __nv_bfloat16 w = row[cache_idx[pi]];
                const double wd = bf16_to_double(w);
                const int q8 = quantize_code(wd, s8, m8, HI_BITS);
                const int qb = quantize_code(wd, sb, mb, base_bits);
                const long long o = (long long)pi * d + n;
                ex.q8[o] = (uint8_t)q8;
                ex.cache_w[o] = w;
                ex.delta[o] = __double2half((s8 * (double)q8 + m8) - (sb * (double)qb + mb));
                ++pi;
            }
        }
    }
}

// Code and difference of cached channel (pool position pi, hidden unit c) in output row n, from the bf16 original:
// target parameters (s, m) given, base parameters from the group's extrema.
__device__ __forceinline__ void down_requant_one(const DownExpertDev& ex, int d, int ng, int G, int n, int pi, int c,
                                                 double s, double m, int hi_bits, int base_bits) {
    const uint32_t mm = ex.gminmax[(long long)n * ng + c / G];
    const double lo = bf16_to_double(__ushort_as_bfloat16((unsigned short)(mm & 0xffff)));
    const double hi = bf16_to_double(__ushort_as_bfloat16((unsigned short)(mm >> 16)));
    __half s_h, m_h;
    double sb, mb;
    group_params(lo, hi, base_bits, s_h, m_h, sb, mb);
    const double wd = bf16_to_double(ex.cache_w[(long long)pi * d + n]);
    const int q = quantize_code(wd, s, m, hi_bits);
    const int qb = quantize_code(wd, sb, mb, base_bits);
    ex.q8[(long long)pi * d + n] = (uint8_t)q;
    ex.delta[(long long)pi * d + n] = __double2half((s * (double)q + m) - (sb * (double)qb + mb));
}

// Another target precision for the cached channels of one expert: one thread per output row n.
__global__ void retarget_down_kernel(int d, int f, int G, int P2, const int32_t* __restrict__ cache_idx, int base_bits,
                                     int hi_bits, DownExpertDev ex) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= d) return;
    const int ng = f / G;
    int pi = 0;
    for (int g = 0; g < ng; ++g) {
        const uint32_t mm = ex.gminmax[(long long)n * ng + g];
        const double lo = bf16_to_double(__ushort_as_bfloat16((unsigned short)(mm & 0xffff)));
        const double hi = bf16_to_double(__ushort_as_bfloat16((unsigned short)(mm >> 16)));
        __half s_h, m_h;
        double s, m;
        group_params(lo, hi, hi_bits, s_h, m_h, s, m);
        __half2 pr = __halves2half2(s_h, m_h);
        ex.s8m8[(long long)n * ng + g] = *reinterpret_cast<uint32_t*>(&pr);
        for (; pi < P2 && cache_idx[pi] < (g + 1) * G; ++pi)
            down_requant_one(ex, d, ng, G, n, pi, cache_idx[pi], s, m, hi_bits, base_bits);
    }
}

// Channel replacement followed by requantization for the set just installed (its tables are already on the device in
// stream order): grid (rows, experts); codes and differences of the set's channels at the expert's target precision.
__global__ void requant_down_kernel(const LayerDev* __restrict__ L, const DownDev* __restrict__ D2,
                                    const int32_t* __restrict__ hi_bits) {
    const int e = blockIdx.y;
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= L->d || !L->ex[e].switchable) return;
    const DownExpertDev& ex = D2->ex[e];
    const int ng = L->f / L->G, S2 = D2->S2, cnt = D2->sig_cnt[e];
    for (int i = 0; i < cnt; ++i) {
        const int c = D2->sig_chan[(long long)e * S2 + i], pi = D2->sig_pool[(long long)e * S2 + i];
        const uint32_t prw = ex.s8m8[(long long)n * ng + c / L->G];
        const __half2 pr = *reinterpret_cast<const __half2*>(&prw);
        down_requant_one(ex, L->d, ng, L->G, n, pi, c, (double)__low2float(pr), (double)__high2float(pr), hi_bits[e],
                         L->ex[e].bits);
    }
}

constexpr int FIX_ROWS = 8;       // one 8-row group of physical rows per CTA (segments start at multiples of 8)
constexpr int FIX_THREADS = 256;
constexpr int FIX_MAX_SIG = 256;  // capacity of a significant set

// grid (row groups, d / (512 / KS)), 256 threads = (256 / KS) adjacent column pairs x KS slices of the set.
// h of the group's rows at the expert's significant hidden units goes to shared memory (unscaled: the buffer holds h
// times a power of two that depends on the base bit-width and the position); every thread accumulates its two
// output columns over its slice of the set (differences loaded eight slots ahead: independent loads), the slices
// are summed through shared memory and added to the down GEMM's result.  KS = 4 for decode-sized batches, where
// the kernel is a chain of memory latencies and more, shorter chains run in parallel; 1 otherwise.
template <int KS>
__global__ void __launch_bounds__(FIX_THREADS) down_fix_kernel(const LayerDev* __restrict__ L,
                                                               const DownDev* __restrict__ D2, WsDev ws) {
    constexpr int PAIRS = FIX_THREADS / KS;
    __shared__ __align__(16) float hs[FIX_MAX_SIG][FIX_ROWS];
    __shared__ int pl[FIX_MAX_SIG], ch[FIX_MAX_SIG];
    __shared__ float red[KS > 1 ? (KS - 1) * FIX_ROWS * 2 * PAIRS : 1];
    pdl_prologue();
    const int row0 = blockIdx.x * FIX_ROWS;
    if (row0 >= ws.off_pad[L->E + L->Es]) return;
    const int e = ws.row_expert[row0];
    if (e < 0 || e >= L->E || !L->ex[e].switchable) return;
    const int cnt = min(D2->sig_cnt[e], FIX_MAX_SIG);
    const int n_e = ws.counts[e];
    const int nrows = min(FIX_ROWS, ws.off_pad[e] + n_e - row0);
    if (cnt <= 0 || nrows <= 0) return;
    const bool tile_layout = n_e > ws.tc_min;  // which FFN kernel wrote this expert's h
    const int bits = L->ex[e].bits, S2 = D2->S2, d = L->d;
    for (int i = threadIdx.x; i < cnt; i += FIX_THREADS) {
        pl[i] = D2->sig_pool[(long long)e * S2 + i];
        ch[i] = D2->sig_chan[(long long)e * S2 + i];
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < FIX_ROWS * cnt; idx += FIX_THREADS) {
        const int i = idx / FIX_ROWS, r = idx - i * FIX_ROWS;
        float v = 0.f;
        if (r < nrows) {
            const int c = ch[i], kc = c >> 7, kk = c & 127;
            const uint8_t* p = tile_layout
                                   ? ws.hbuf + act_off(kc, row0, ws.Rcap) + ((kk >> 3) * 8 + r) * 16 + (kk & 7) * 2
                                   : ws.hbuf + act_off(kc, row0 + r, ws.Rcap) + kk * 2;
            const float unscale = __uint_as_float((uint32_t)(127 - x_scale_exp(bits, kk)) << 23);
            v = __half2float(*reinterpret_cast<const __half*>(p)) * unscale;
        }
        hs[i][r] = v;
    }
    __syncthreads();
    const int cp = threadIdx.x % PAIRS, ks = threadIdx.x / PAIRS;
    const int n = (blockIdx.y * PAIRS + cp) * 2;
    const bool col_ok = n < d;
    const __half* dl = D2->ex[e].delta + n;
    const int per = (cnt + KS - 1) / KS;
    const int i_beg = ks * per, i_end = min(cnt, i_beg + per);
    float acc[FIX_ROWS][2];
#pragma unroll
    for (int r = 0; r < FIX_ROWS; ++r) acc[r][0] = acc[r][1] = 0.f;
    if (col_ok) {
        for (int i0 = i_beg; i0 < i_end; i0 += 8) {
            __half2 w[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
                w[j] = (i0 + j < i_end) ? *reinterpret_cast<const __half2*>(dl + (long long)pl[i0 + j] * d)
                                        : __float2half2_rn(0.f);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (i0 + j >= i_end) break;
                const float2 wf = __half22float2(w[j]);
                const float4 ha = *reinterpret_cast<const float4*>(&hs[i0 + j][0]);
                const float4 hb = *reinterpret_cast<const float4*>(&hs[i0 + j][4]);
                const float hr[8] = {ha.x, ha.y, ha.z, ha.w, hb.x, hb.y, hb.z, hb.w};
#pragma unroll
                for (int r = 0; r < FIX_ROWS; ++r) {
                    acc[r][0] = fmaf(hr[r], wf.x, acc[r][0]);
                    acc[r][1] = fmaf(hr[r], wf.y, acc[r][1]);
                }
            }
        }
    }
    if constexpr (KS > 1) {
        if (ks > 0) {
#pragma unroll
            for (int r = 0; r < FIX_ROWS; ++r) {
                red[(((ks - 1) * FIX_ROWS + r) * 2 + 0) * PAIRS + cp] = acc[r][0];
                red[(((ks - 1) * FIX_ROWS + r) * 2 + 1) * PAIRS + cp] = acc[r][1];
            }
        }
        __syncthreads();
        if (ks > 0) return;
#pragma unroll
        for (int g = 0; g < KS - 1; ++g)  // slices are added in slice order: the result does not depend on timing
#pragma unroll
            for (int r = 0; r < FIX_ROWS; ++r) {
                acc[r][0] += red[((g * FIX_ROWS + r) * 2 + 0) * PAIRS + cp];
                acc[r][1] += red[((g * FIX_ROWS + r) * 2 + 1) * PAIRS + cp];
            }
    }
    if (!col_ok) return;
#pragma unroll
    for (int r = 0; r < FIX_ROWS; ++r)
        if (r < nrows) {  // K split 0; the combine adds the splits
            float2* y = reinterpret_cast<float2*>(ws.ypart + (long long)(row0 + r) * d + n);
            float2 v = *y;
            v.x += acc[r][0];
            v.y += acc[r][1];
            *y = v;
        }
}

// Logical 8-bit codes [d][f] (0 outside the cached / the significant channels) and parameters [d][f/G].
__global__ void export_down_kernel(const LayerDev* __restrict__ L, const DownDev* __restrict__ D2, int e, int which,
                                   uint8_t* __restrict__ q, uint16_t* __restrict__ sc, uint16_t* __restrict__ zr) {
    const int d = L->d, f = L->f, G = L->G, ng = f / G;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)d * f) return;
    const int n = (int)(idx / f), k = (int)(idx % f);
    const int P2 = D2->P2, S2 = D2->S2;
    const int32_t* ci = D2->cache_idx + (long long)e * P2;
    int lo = 0, hi = P2 - 1, p = -1;
    while (lo <= hi) {
        const int mid = (lo + hi) >> 1, v = ci[mid];
        if (v == k) { p = mid; break; }
        if (v < k) lo = mid + 1; else hi = mid - 1;
    }
    bool take = p >= 0;
    if (take && which == 2) {
        take = false;
        const int cnt = D2->sig_cnt[e];
        for (int i = 0; i < cnt; ++i) take = take || D2->sig_chan[(long long)e * S2 + i] == k;
    }
    q[idx] = take ? D2->ex[e].q8[(long long)p * d + n] : (uint8_t)0;
    if (k % G == 0) {
        const uint32_t prw = D2->ex[e].s8m8[(long long)n * ng + k / G];
        sc[(long long)n * ng + k / G] = (uint16_t)(prw & 0xffff);
        zr[(long long)n * ng + k / G] = (uint16_t)(prw >> 16);
    }
}

cudaError_t launch_pack_down_hi(const void* w_down, int d, int f, int G, int P2, const int32_t* cache_idx_dev,
                                int base_bits, const DownExpertDev& ex, cudaStream_t st) {
    pack_down_hi_kernel<<<(d + 127) / 128, 128, 0, st>>>((const __nv_bfloat16*)w_down, d, f, G, P2, cache_idx_dev,
                                                         base_bits, ex);
    return cudaGetLastError();
}

cudaError_t launch_retarget_down(int d, int f, int G, int P2, const int32_t* cache_idx_dev, int base_bits, int hi_bits,
                                 const DownExpertDev& ex, cudaStream_t st) {
    retarget_down_kernel<<<(d + 127) / 128, 128, 0, st>>>(d, f, G, P2, cache_idx_dev, base_bits, hi_bits, ex);
    return cudaGetLastError();
}

cudaError_t launch_requant_down(const LayerDev* L, const DownDev* D2, const int32_t* hi_bits_dev, int d, int n_experts,
                                cudaStream_t st) {
    requant_down_kernel<<<dim3((unsigned)((d + 127) / 128), (unsigned)n_experts), 128, 0, st>>>(L, D2, hi_bits_dev);
    return cudaGetLastError();
}

cudaError_t launch_down_fix(const LayerDev* L, const DownDev* D2, const WsDev& ws, int d, cudaStream_t st) {
    const unsigned groups = (unsigned)((ws.Rpad + FIX_ROWS - 1) / FIX_ROWS);
    if (ws.R <= 512) {  // decode-sized: four slices of the set per column pair, four times the CTAs
        const dim3 grid(groups, (unsigned)((d + 127) / 128));
        return launch_pdl(down_fix_kernel<4>, grid, dim3(FIX_THREADS), 0, st, L, D2, ws);
    }
    const dim3 grid(groups, (unsigned)((d + 511) / 512));
    return launch_pdl(down_fix_kernel<1>, grid, dim3(FIX_THREADS), 0, st, L, D2, ws);
}

cudaError_t launch_export_down(const LayerDev* L, const DownDev* D2, int e, int which, long long n_elems, uint8_t* q,
                               uint16_t* sc, uint16_t* zr, cudaStream_t st) {
    export_down_kernel<<<(unsigned)((n_elems + 255) / 256), 256, 0, st>>>(L, D2, e, which, q, sc, zr);
    return cudaGetLastError();
}

}  // namespace dyn
