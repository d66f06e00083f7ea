// Offline quantize + bit-pack kernels and their inverse (export of logical codes).
//
// Quantizer (per row, per group of G consecutive input indices), all in IEEE double:
//   scale = fp16((max - min) / (2^b - 1))  (1.0 if that rounds to 0),  zero = fp16(min),
//   code  = clamp(rint((w - zero) / scale), 0, 2^b - 1)   (true division, ties to even).
// The double -> fp16 conversions are single roundings (cvt.rn.f16.f64).
#include "common.cuh"
#include "layout.cuh"
#include "quant.cuh"

namespace dyn {

// One CTA packs one block (256 rows x 128 k).  Thread r owns row r of the block.
// src_a / src_b: row-major [rows_src, K] bf16; for the fused gate/up matrix (fused = 1) rows 0..7 of
// every atom come from src_a (gate) and rows 8..15 from src_b (up); otherwise only src_a is used.
__global__ void __launch_bounds__(256) pack_blocks_kernel(const __nv_bfloat16* __restrict__ src_a,
                                                          const __nv_bfloat16* __restrict__ src_b, int K, int G,
                                                          int bits, int fused, uint8_t* __restrict__ dst,
                                                          int blk_bytes, int n_kc) {
    extern __shared__ __align__(16) uint32_t sm_words[];  // packed codes of the block, then params
    const int kc = blockIdx.x, rb = blockIdx.y, r = threadIdx.x;
    const int code_words = block_code_bytes(bits) / 4;
    const int ngrp = KC / G;
    for (int i = r; i < code_words; i += 256) sm_words[i] = 0;
    __syncthreads();

    const int atom = r >> 4, ra = r & 15;
    const __nv_bfloat16* src;
    long long row;
    if (fused) {
        src = (ra < 8) ? src_a : src_b;
        row = w13_hidden_index(rb, r);
    } else {
        src = src_a;
        row = (long long)rb * RB + r;
    }
    const __nv_bfloat16* p = src + row * K + (long long)kc * KC;
    uint32_t* atom_words = sm_words + atom * (atom_bytes(bits) / 4);
    for (int g = 0; g < ngrp; ++g) {
        double lo = bf16_to_double(p[g * G]), hi = lo;
        for (int i = 1; i < G; ++i) {
            double v = bf16_to_double(p[g * G + i]);
            lo = v < lo ? v : lo;
            hi = v > hi ? v : hi;
        }
        __half s_h, m_h;
        double s, m;
        group_params(lo, hi, bits, s_h, m_h, s, m);
        __half2 pr = __halves2half2(s_h, m_h);
        sm_words[code_words + r * ngrp + g] = *reinterpret_cast<uint32_t*>(&pr);
        for (int i = 0; i < G; ++i) {
            const int kk = g * G + i;
            const int q = quantize_code(bf16_to_double(p[kk]), s, m, bits);
            if (bits == 3 || bits == 6) {   // two bit planes: the low 2 (4) bits and the high 1 (2) bits
                const int lowb = bits == 3 ? 2 : 4;
                CodeLoc a = code_loc(bits, ra, kk, 0), b = code_loc(bits, ra, kk, 1);
                atomicOr(&atom_words[a.byte_off >> 2], (uint32_t)(q & ((1 << lowb) - 1)) << a.shift);
                atomicOr(&atom_words[b.byte_off >> 2], (uint32_t)(q >> lowb) << b.shift);
            } else {
                CodeLoc a = code_loc(bits, ra, kk, 0);
                atomicOr(&atom_words[a.byte_off >> 2], (uint32_t)q << a.shift);
            }
        }
    }
    __syncthreads();
    uint32_t* out = reinterpret_cast<uint32_t*>(dst + ((long long)rb * n_kc + kc) * blk_bytes);
    for (int i = r; i < blk_bytes / 4; i += 256) out[i] = sm_words[i];
}

// 8-bit side data of a switchable expert, one thread per row n of one matrix (mat 0 = gate, 1 = up):
// the 8-bit params of every group, and for each cached channel its 8-bit code, its bf16 original
// (the channel cache) and the forward-ready fp16 value s8*q8 + m8.
__global__ void pack_hi_kernel(const __nv_bfloat16* __restrict__ w_gate, const __nv_bfloat16* __restrict__ w_up,
                               int f, int d, int G, int P, const int32_t* __restrict__ cache_idx, ExpertDev ex) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int mat = blockIdx.y;
    if (n >= f) return;
    const __nv_bfloat16* row = (mat ? w_up : w_gate) + (long long)n * d;
    const int ng = d / G;
    const int rb = n >> 7, rib = w13_row_in_block(n, mat);
    int pi = 0;
    for (int g = 0; g < ng; ++g) {
        double lo = bf16_to_double(row[g * G]), hi = lo;
        __nv_bfloat16 lo_b = row[g * G], hi_b = lo_b;
        for (int i = 1; i < G; ++i) {
            double v = bf16_to_double(row[g * G + i]);
            if (v < lo) { lo = v; lo_b = row[g * G + i]; }
            if (v > hi) { hi = v; hi_b = row[g * G + i]; }
        }
        // the group's extrema stay with the cache: a later change of the target precision needs them
        ex.gminmax[mat][(long long)n * ng + g] =
            (uint32_t)__bfloat16_as_ushort(lo_b) | ((uint32_t)__bfloat16_as_ushort(hi_b) << 16);
        __half s_h, m_h;
        double s, m;
        group_params(lo, hi, HI_BITS, s_h, m_h, s, m);
        __half2 pr = __halves2half2(s_h, m_h);
        ex.s8m8[mat][(long long)n * ng + g] = *reinterpret_cast<uint32_t*>(&pr);
        while (pi < P && cache_idx[pi] < (g + 1) * G) {
            const int c = cache_idx[pi];
            const __nv_bfloat16 w = row[c];
            const int q = quantize_code(bf16_to_double(w), s, m, HI_BITS);
            ex.pool_q8[mat][(long long)pi * f + n] = (uint8_t)q;
            ex.cache_w[mat][(long long)pi * f + n] = w;
            ex.pool_hi[pool_tile_off(rb, pi, (P + 31) & ~31) / 2 + rib] = __double2half(s * (double)q + m);
            ++pi;
        }
    }
}

// Re-derive the 8-bit codes (and forward-ready values) of selected cached channels from the bf16
// originals in the channel cache: channel replacement followed by requantization.
// list: [n_items] packed (expert << 16 | pool position); grid.x covers rows, grid.y = items, grid.z = mat.
__global__ void requant_from_cache_kernel(const LayerDev* __restrict__ L, const int32_t* __restrict__ items) {
    const int item = items[blockIdx.y];
    const int e = item >> 16, p = item & 0xffff;
    const int mat = blockIdx.z;
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const ExpertDev& ex = L->ex[e];
    if (n >= L->f || !ex.switchable) return;
    const int c = L->cache_idx[e * L->P + p];
    const int ng = L->d / L->G;
    const uint32_t prw = ex.s8m8[mat][(long long)n * ng + c / L->G];
    const __half2 pr = *reinterpret_cast<const __half2*>(&prw);
    const double s = (double)__low2float(pr), m = (double)__high2float(pr);
    const __nv_bfloat16 w = ex.cache_w[mat][(long long)p * L->f + n];
    const int q = quantize_code(bf16_to_double(w), s, m, ex.hi_bits);
    ex.pool_q8[mat][(long long)p * L->f + n] = (uint8_t)q;
    const int rb = n >> 7, rib = w13_row_in_block(n, mat);
    ex.pool_hi[pool_tile_off(rb, p, L->P_pad) / 2 + rib] = __double2half(s * (double)q + m);
}

// Change the precision the cached channels of expert e are served at (Section IV-B: after replacement the
// original channels are requantized to the precision the new data calls for, higher or lower than before):
// the parameters of every group at `bits` from the stored group extrema, then code and forward-ready value of
// every cached channel from its bf16 original.  One thread per row n of one matrix (grid.y: gate, up).
__global__ void retarget_kernel(LayerDev* __restrict__ L, int e, int bits) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int mat = blockIdx.y;
    ExpertDev& ex = L->ex[e];
    if (n == 0 && mat == 0) ex.hi_bits = bits;
    if (n >= L->f) return;
    const int ng = L->d / L->G, G = L->G, P = L->P, f = L->f;
    const int32_t* ci = L->cache_idx + (long long)e * P;
    const int rb = n >> 7, rib = w13_row_in_block(n, mat);
    int pi = 0;
    for (int g = 0; g < ng; ++g) {
        const uint32_t mm = ex.gminmax[mat][(long long)n * ng + g];
        const double lo = bf16_to_double(__ushort_as_bfloat16((unsigned short)(mm & 0xffff)));
        const double hi = bf16_to_double(__ushort_as_bfloat16((unsigned short)(mm >> 16)));
        __half s_h, m_h;
        double s, m;
        group_params(lo, hi, bits, s_h, m_h, s, m);
        __half2 pr = __halves2half2(s_h, m_h);
        ex.s8m8[mat][(long long)n * ng + g] = *reinterpret_cast<uint32_t*>(&pr);
        while (pi < P && ci[pi] < (g + 1) * G) {
            const __nv_bfloat16 w = ex.cache_w[mat][(long long)pi * f + n];
            const int q = quantize_code(bf16_to_double(w), s, m, bits);
            ex.pool_q8[mat][(long long)pi * f + n] = (uint8_t)q;
            ex.pool_hi[pool_tile_off(rb, pi, L->P_pad) / 2 + rib] = __double2half(s * (double)q + m);
            ++pi;
        }
    }
}

// Export logical codes and params.  One thread per (n, k).
__global__ void export_kernel(const LayerDev* __restrict__ L, int e, int mat, int which, uint8_t* __restrict__ q,
                              uint16_t* __restrict__ sc, uint16_t* __restrict__ zr) {
    const int K = (mat == 2) ? L->f : L->d;
    const int N = (mat == 2) ? L->d : L->f;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)N * K) return;
    const int n = (int)(idx / K), k = (int)(idx % K);
    const ExpertDev& ex = L->ex[e];
    const int G = L->G, ng = K / G;
    if (which == 0) {
        const int bits = ex.bits;
        int rb, r, n_kc;
        const uint8_t* base;
        if (mat == 2) { rb = n / RB; r = n % RB; n_kc = L->n_kc2; base = ex.w2; }
        else { rb = n >> 7; r = w13_row_in_block(n, mat); n_kc = L->n_kc13; base = ex.w13; }
        const int kc = k / KC, kk = k % KC;
        const uint8_t* blk = base + ((long long)rb * n_kc + kc) * ex.blk_bytes;
        const uint8_t* atom = blk + (r >> 4) * atom_bytes(bits);
        int code;
        if (bits == 3 || bits == 6) {
            const int lowb = bits == 3 ? 2 : 4;
            CodeLoc a = code_loc(bits, r & 15, kk, 0), b = code_loc(bits, r & 15, kk, 1);
            const uint32_t wa = *reinterpret_cast<const uint32_t*>(atom + a.byte_off);
            const uint32_t wb = *reinterpret_cast<const uint32_t*>(atom + b.byte_off);
            code = ((wa >> a.shift) & ((1u << lowb) - 1)) | (((wb >> b.shift) & ((1u << (bits - lowb)) - 1)) << lowb);
        } else {
            CodeLoc a = code_loc(bits, r & 15, kk, 0);
            const uint32_t wa = *reinterpret_cast<const uint32_t*>(atom + a.byte_off);
            code = (wa >> a.shift) & ((1u << bits) - 1);
        }
        q[idx] = (uint8_t)code;
        if (kk % G == 0) {
            const uint32_t prw =
                *reinterpret_cast<const uint32_t*>(blk + block_code_bytes(bits) + (r * (KC / G) + kk / G) * 4);
            sc[(long long)n * ng + k / G] = (uint16_t)(prw & 0xffff);
            zr[(long long)n * ng + k / G] = (uint16_t)(prw >> 16);
        }
    } else {
        // binary search of k in the expert's cache headers
        const int32_t* ci = L->cache_idx + e * L->P;
        int lo = 0, hi = L->P - 1, p = -1;
        while (lo <= hi) {
            int mid = (lo + hi) >> 1;
            int v = ci[mid];
            if (v == k) { p = mid; break; }
            if (v < k) lo = mid + 1; else hi = mid - 1;
        }
        bool take = p >= 0;
        if (which == 2 && take) take = (L->sigmask[e * (L->d / 32) + (k >> 5)] >> (k & 31)) & 1u;
        q[idx] = take ? ex.pool_q8[mat][(long long)p * L->f + n] : (uint8_t)0;
        if (k % G == 0) {
            const uint32_t prw = ex.s8m8[mat][(long long)n * ng + k / G];
            sc[(long long)n * ng + k / G] = (uint16_t)(prw & 0xffff);
            zr[(long long)n * ng + k / G] = (uint16_t)(prw >> 16);
        }
    }
}

// ---- host launchers ----------------------------------------------------------------------

cudaError_t launch_pack_blocks(const void* src_a, const void* src_b, int n_rows_blocks, int K, int G, int bits,
                               int fused, void* dst, cudaStream_t st) {
    const int blk = block_bytes(bits, G);
    dim3 grid(K / KC, n_rows_blocks);
    cudaError_t err = cudaFuncSetAttribute(pack_blocks_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, blk);
    if (err != cudaSuccess) return err;
    pack_blocks_kernel<<<grid, 256, blk, st>>>((const __nv_bfloat16*)src_a, (const __nv_bfloat16*)src_b, K, G, bits,
                                               fused, (uint8_t*)dst, blk, K / KC);
    return cudaGetLastError();
}

cudaError_t launch_pack_hi(const void* w_gate, const void* w_up, int f, int d, int G, int P,
                           const int32_t* cache_idx_dev, const ExpertDev& ex, cudaStream_t st) {
    dim3 grid((f + 127) / 128, 2);
    pack_hi_kernel<<<grid, 128, 0, st>>>((const __nv_bfloat16*)w_gate, (const __nv_bfloat16*)w_up, f, d, G, P,
                                         cache_idx_dev, ex);
    return cudaGetLastError();
}

cudaError_t launch_retarget(LayerDev* L, int e, int f, int bits, cudaStream_t st) {
    dim3 grid((f + 127) / 128, 2);
    retarget_kernel<<<grid, 128, 0, st>>>(L, e, bits);
    return cudaGetLastError();
}

cudaError_t launch_requant(const LayerDev* L, int f, const int32_t* items_dev, int n_items, cudaStream_t st) {
    if (n_items <= 0) return cudaSuccess;
    dim3 grid((f + 255) / 256, n_items, 2);
    requant_from_cache_kernel<<<grid, 256, 0, st>>>(L, items_dev);
    return cudaGetLastError();
}

cudaError_t launch_export(const LayerDev* L, int e, int mat, int which, long long n_elems, uint8_t* q, uint16_t* sc,
                          uint16_t* zr, cudaStream_t st) {
    const int threads = 256;
    const long long blocks = (n_elems + threads - 1) / threads;
    export_kernel<<<(unsigned)blocks, threads, 0, st>>>(L, e, mat, which, q, sc, zr);
    return cudaGetLastError();
}

}  // namespace dyn
