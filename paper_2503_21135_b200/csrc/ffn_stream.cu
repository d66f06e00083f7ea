// Streaming grouped dequant-GEMM for small token counts per expert (decode path, and the generic
// fallback for any size): HBM-bound, judged on packed-weight bytes per second.
//
// One CTA = one (expert, 256-row weight block, chunk of <= 32 tokens, K split).  A producer warp
// streams the packed blocks (codes + params, contiguous per 256 x 128 block) and the matching
// activation slices into a shared-memory ring with bulk async copies completing on mbarriers; eight
// consumer warps, each owning two 16-row atoms, turn codes into fp16 operands with ONE logic op per
// register pair: a code field masked in place at bit offset o is the fp16 subnormal q * 2^(o-24),
// and the activation slice already carries the factor 2^(bias-o) (see layout.cuh).  They issue
// mma.sync m16n8k16 (weights = A, tokens = B, fp32 accumulate) and apply scale / zero once per
// group after the dot product:
//     sum_k (s*q_k + m) x_k = (s * 2^(24-bias)) * acc + m * sum_k x_k .
// The per-group sums of x come precomputed with the activation slice.  Codes and activations are
// exact in fp16, so the only roundings are the fp32 accumulation and the fp16 rounding of h.
// The number of 8-token tiles (1..4) is chosen per CTA from the expert's actual token count.
//
// Gate/up variant: after the K loop the significant-channel correction runs as extra ring stages
// (16 channels each): the fp16 tiles of the active cached channels are fetched through the slot ->
// pool-position table and multiplied with the gathered activation columns into the same
// accumulators; then SwiGLU, fp16 rounding of h, per-64 sums of h, coalesced store of h (scaled
// for the down matrix).  Down variant: writes fp32 partial outputs per K split.
#include <type_traits>

#include "common.cuh"
#include "expand.cuh"
#include "layout.cuh"

namespace dyn {

constexpr int CONSUMER_WARPS = 8;
constexpr int FFN_THREADS = (CONSUMER_WARPS + 1) * 32;
constexpr int SIG_TILE_STRIDE = 528;  // 512 B tile + 16 B pad: conflict-free ldmatrix rows
constexpr int SIG_X_STRIDE = 48;      // 32 B of gathered activations per token + pad
constexpr int SMEM_HEADER = 256;
constexpr int MAX_STAGES = 8;
constexpr int CHUNK_TOKENS = 32;

__host__ __device__ inline int stage_bytes_for(int bits, int G, int NT) {
    const int b = block_bytes(bits, G) + NT * XROW;
    return (b + 127) & ~127;
}

struct FfnParams {
    const LayerDev* L;
    WsDev ws;
    int n_tc;          // token chunks per expert launched (grid.x = n_tc * n_rb * ksplit)
    int ksplit;
    long long split_stride;  // elements between K-split partial outputs
    int smem_bytes;
};

template <int BITS, int NT8, bool GATEUP>
__device__ __forceinline__ void ffn_body(const FfnParams& p, const ExpertDev& ex, int e, int rb, int split, int row0,
                                         int nvalid, uint8_t* smem) {
    constexpr int NT = NT8 * 8;
    const LayerDev* L = p.L;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = L->G;
    const int K = GATEUP ? L->d : L->f;
    const int n_kc = K / KC;
    const int blk_bytes = ex.blk_bytes;
    const int code_bytes = block_code_bytes(BITS);
    const int stage_bytes = stage_bytes_for(BITS, G, NT);
    const int htile_bytes = GATEUP ? NT * XROW : 0;
    int NS = (p.smem_bytes - SMEM_HEADER - htile_bytes) / stage_bytes;
    NS = NS > MAX_STAGES ? MAX_STAGES : NS;

    uint64_t* full = reinterpret_cast<uint64_t*>(smem);
    uint64_t* empty = full + MAX_STAGES;
    uint64_t* done = empty + MAX_STAGES;
    volatile int* poison = reinterpret_cast<volatile int*>(smem + (2 * MAX_STAGES + 1) * 8);
    uint8_t* stages = smem + SMEM_HEADER;
    uint8_t* htile = stages + (size_t)NS * stage_bytes;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], CONSUMER_WARPS);
        }
        mbar_init(done, CONSUMER_WARPS);
        *poison = 0;
        fence_barrier_init();
    }
    __syncthreads();

    int kc0 = 0, kc1 = n_kc;
    if (!GATEUP) {
        kc0 = (int)(((long long)split * n_kc) / p.ksplit);
        kc1 = (int)(((long long)(split + 1) * n_kc) / p.ksplit);
    }
    const bool do_sig = GATEUP && ex.switchable && (L->sig_cnt[e] > 0);
    const int n_ss = do_sig ? (L->sig_cnt[e] + 15) / 16 : 0;
    const uint8_t* wbase = (GATEUP ? ex.w13 : ex.w2) + (size_t)rb * n_kc * blk_bytes;
    const uint8_t* xbase = (GATEUP ? p.ws.xperm : p.ws.hbuf) + (size_t)row0 * n_kc * XROW;

    if (warp == CONSUMER_WARPS) {
        // ---------------- producer warp ----------------
        int it = 0;
        bool ok = true;
        for (int kc = kc0; kc < kc1 && ok; ++kc, ++it) {
            const int s = it % NS, ph = (it / NS) & 1;
            int okl = 1;
            if (lane == 0) okl = mbar_wait_bounded(&empty[s], ph ^ 1, poison, p.ws.status) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, okl, 0) != 0;
            if (!ok) break;
            uint8_t* st = stages + (size_t)s * stage_bytes;
            if (lane == 0) {
                mbar_arrive_expect_tx(&full[s], (uint32_t)(blk_bytes + nvalid * XROW));
                bulk_g2s(st, wbase + (size_t)kc * blk_bytes, (uint32_t)blk_bytes, &full[s]);
            }
            __syncwarp();
            if (lane < nvalid)
                bulk_g2s(st + blk_bytes + lane * XROW, xbase + ((size_t)lane * n_kc + kc) * XROW, XROW, &full[s]);
        }
        if constexpr (GATEUP) {
            const int S_pad = L->S_pad;
            for (int ss = 0; ss < n_ss && ok; ++ss, ++it) {
                const int s = it % NS, ph = (it / NS) & 1;
                int okl = 1;
                if (lane == 0) okl = mbar_wait_bounded(&empty[s], ph ^ 1, poison, p.ws.status) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, okl, 0) != 0;
                if (!ok) break;
                uint8_t* st = stages + (size_t)s * stage_bytes;
                if (lane == 0) mbar_arrive_expect_tx(&full[s], (uint32_t)(16 * POOL_TILE_BYTES + nvalid * 32));
                __syncwarp();
                if (lane < 16) {
                    const int pos = L->sig_pool[e * S_pad + ss * 16 + lane];
                    bulk_g2s(st + lane * SIG_TILE_STRIDE, ex.pool_hi + ((size_t)rb * (L->P + 1) + pos) * RB,
                             POOL_TILE_BYTES, &full[s]);
                }
                if (lane < nvalid)
                    bulk_g2s(st + 16 * SIG_TILE_STRIDE + lane * SIG_X_STRIDE,
                             p.ws.xsig + (size_t)(row0 + lane) * S_pad + ss * 16, 32, &full[s]);
            }
        }
        if (!ok && lane == 0) {
            // gave up: let copies already issued land before the CTA's shared memory is released
            const unsigned long long t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 2000000ull) {
            }
        }
        return;
    }

    // ---------------- consumer warps ----------------
    const int gid = lane >> 2, tid4 = lane & 3;
    const int atom0 = warp * 2;
    float total[2][NT8][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int j = 0; j < NT8; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) total[a][j][c] = 0.f;

    // exact power of two that undoes the operand scaling: codes enter as q*2^(o-24), activations as x*2^(bias-o)
    const float unscale = __uint_as_float((uint32_t)(127 + 24 - x_scale_bias(BITS)) << 23);

    int it = 0;
    bool ok = true;
    for (int kc = kc0; kc < kc1; ++kc, ++it) {
        const int s = it % NS, ph = (it / NS) & 1;
        ok = mbar_wait_bounded(&full[s], ph, poison, p.ws.status);
        if (!ok) break;
        const uint8_t* st = stages + (size_t)s * stage_bytes;
        const uint8_t* xs = st + blk_bytes;
        const uint32_t* prm = reinterpret_cast<const uint32_t*>(st + code_bytes);
        const int ngrp = KC / G;
        float accg[2][NT8][4];
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int j = 0; j < NT8; ++j)
#pragma unroll
                for (int c = 0; c < 4; ++c) accg[a][j][c] = 0.f;

#pragma unroll
        for (int half = 0; half < 2; ++half) {
            Codes<BITS> cd[2];
#pragma unroll
            for (int a = 0; a < 2; ++a) load_codes<BITS>(cd[a], st + (atom0 + a) * atom_bytes(BITS), lane, half);

            auto step = [&](auto S4c) {
                constexpr int S4 = decltype(S4c)::value;
                const int sidx = half * 4 + S4;
                uint32_t b0[NT8], b1[NT8];
#pragma unroll
                for (int j = 0; j < NT8; ++j) {
                    const uint2 v =
                        *reinterpret_cast<const uint2*>(xs + (8 * j + gid) * XROW + (16 * sidx + 4 * tid4) * 2);
                    b0[j] = v.x;
                    b1[j] = v.y;
                }
#pragma unroll
                for (int a = 0; a < 2; ++a) {
                    uint32_t af[4];
                    expand<BITS, S4>(cd[a], af);
#pragma unroll
                    for (int j = 0; j < NT8; ++j) mma16816(accg[a][j], af, b0[j], b1[j]);
                }
            };
            step(std::integral_constant<int, 0>{});
            step(std::integral_constant<int, 1>{});
            step(std::integral_constant<int, 2>{});
            step(std::integral_constant<int, 3>{});

            if (G == 64 || half == 1) {
                const int g = (G == 64) ? half : 0;
#pragma unroll
                for (int a = 0; a < 2; ++a) {
                    const int r0 = (atom0 + a) * 16 + gid;
                    const uint32_t p0 = prm[r0 * ngrp + g], p1 = prm[(r0 + 8) * ngrp + g];
                    const __half2 h0 = *reinterpret_cast<const __half2*>(&p0);
                    const __half2 h1 = *reinterpret_cast<const __half2*>(&p1);
                    const float s0 = __low2float(h0) * unscale, s1 = __low2float(h1) * unscale;
                    const float m0 = __high2float(h0), m1 = __high2float(h1);
#pragma unroll
                    for (int j = 0; j < NT8; ++j) {
                        const float* sp0 =
                            reinterpret_cast<const float*>(xs + (8 * j + 2 * tid4) * XROW + XROW_SUM_OFF);
                        const float* sp1 =
                            reinterpret_cast<const float*>(xs + (8 * j + 2 * tid4 + 1) * XROW + XROW_SUM_OFF);
                        float xs0, xs1;
                        if (G == 64) { xs0 = sp0[half]; xs1 = sp1[half]; }
                        else { xs0 = sp0[0] + sp0[1]; xs1 = sp1[0] + sp1[1]; }
                        total[a][j][0] += fmaf(s0, accg[a][j][0], m0 * xs0);
                        total[a][j][1] += fmaf(s0, accg[a][j][1], m0 * xs1);
                        total[a][j][2] += fmaf(s1, accg[a][j][2], m1 * xs0);
                        total[a][j][3] += fmaf(s1, accg[a][j][3], m1 * xs1);
#pragma unroll
                        for (int c = 0; c < 4; ++c) accg[a][j][c] = 0.f;
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);
    }

    if constexpr (GATEUP) {
        for (int ss = 0; ss < n_ss && ok; ++ss, ++it) {
            const int s = it % NS, ph = (it / NS) & 1;
            ok = mbar_wait_bounded(&full[s], ph, poison, p.ws.status);
            if (!ok) break;
            const uint8_t* st = stages + (size_t)s * stage_bytes;
            const uint8_t* xs = st + 16 * SIG_TILE_STRIDE;
            uint32_t b0[NT8], b1[NT8];
#pragma unroll
            for (int j = 0; j < NT8; ++j) {
                b0[j] = *reinterpret_cast<const uint32_t*>(xs + (8 * j + gid) * SIG_X_STRIDE + (2 * tid4) * 2);
                b1[j] = *reinterpret_cast<const uint32_t*>(xs + (8 * j + gid) * SIG_X_STRIDE + (2 * tid4 + 8) * 2);
            }
            const int mi = lane >> 3, r = lane & 7;
#pragma unroll
            for (int a = 0; a < 2; ++a) {
                uint32_t af[4];
                const uint32_t addr =
                    smem_u32(st + ((mi >> 1) * 8 + r) * SIG_TILE_STRIDE + (16 * (atom0 + a) + (mi & 1) * 8) * 2);
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(af[0]), "=r"(af[1]), "=r"(af[2]), "=r"(af[3])
                             : "r"(addr));
#pragma unroll
                for (int j = 0; j < NT8; ++j) mma16816(total[a][j], af, b0[j], b1[j]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }
    }
    if (!ok) {  // poisoned: drop the outputs (the status word says so); still arrive so nobody waits on us
        __syncwarp();
        if (GATEUP && lane == 0) mbar_arrive(done);
        return;
    }

    if constexpr (GATEUP) {
        // SwiGLU: rows 0..7 of an atom are gate, rows 8..15 the matching up rows.
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int j = 0; j < NT8; ++j)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const float g = total[a][j][c], u = total[a][j][2 + c];
                    const float h = g / (1.f + expf(-g)) * u;
                    const int tok = 8 * j + 2 * tid4 + c;
                    *reinterpret_cast<__half*>(htile + tok * XROW + (8 * (atom0 + a) + gid) * 2) = __float2half_rn(h);
                }
        __syncwarp();
        if (lane == 0) mbar_arrive(done);
        if (!mbar_wait_bounded(done, 0, poison, p.ws.status) || *poison) return;
        const int n_rb = L->n_rb13;  // = chunks of the hidden axis
        // this lane's four hidden indices 4*lane + {0..3}: the down matrix wants them scaled by 2^(bias-o)
        const float sc0 = __uint_as_float((uint32_t)(127 + x_scale_exp(BITS, 4 * lane)) << 23);
        const float sc1 = __uint_as_float((uint32_t)(127 + x_scale_exp(BITS, 4 * lane + 2)) << 23);
        for (int tok = warp; tok < nvalid; tok += CONSUMER_WARPS) {
            const uint2 v = *reinterpret_cast<const uint2*>(htile + tok * XROW + lane * 8);
            const __half2 a2 = *reinterpret_cast<const __half2*>(&v.x), b2 = *reinterpret_cast<const __half2*>(&v.y);
            const float f0 = __low2float(a2), f1 = __high2float(a2), f2 = __low2float(b2), f3 = __high2float(b2);
            float sum = f0 + f1 + f2 + f3;
#pragma unroll
            for (int o = 8; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            const __half2 oa = __floats2half2_rn(f0 * sc0, f1 * sc0), ob = __floats2half2_rn(f2 * sc1, f3 * sc1);
            uint2 ov;
            ov.x = *reinterpret_cast<const uint32_t*>(&oa);
            ov.y = *reinterpret_cast<const uint32_t*>(&ob);
            uint8_t* dst = p.ws.hbuf + ((size_t)(row0 + tok) * n_rb + rb) * XROW;
            *reinterpret_cast<uint2*>(dst + lane * 8) = ov;
            if ((lane & 15) == 0) *reinterpret_cast<float*>(dst + XROW_SUM_OFF + (lane >> 4) * 4) = sum;
        }
    } else {
        float* yb = p.ws.ypart + (size_t)split * p.split_stride;
        const int d = L->d;
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int j = 0; j < NT8; ++j)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int tok = 8 * j + 2 * tid4 + (c & 1);
                    const int n = rb * RB + (atom0 + a) * 16 + gid + ((c >> 1) ? 8 : 0);
                    if (tok < nvalid) yb[(size_t)(row0 + tok) * d + n] = total[a][j][c];
                }
    }
}

template <int BITS, bool GATEUP>
__device__ __forceinline__ void ffn_dispatch_tiles(const FfnParams& p, const ExpertDev& ex, int e, int rb, int split,
                                                   int row0, int nvalid, uint8_t* smem) {
    const int nt8 = (nvalid + 7) >> 3;
    if (nt8 == 1) ffn_body<BITS, 1, GATEUP>(p, ex, e, rb, split, row0, nvalid, smem);
    else if (nt8 == 2) ffn_body<BITS, 2, GATEUP>(p, ex, e, rb, split, row0, nvalid, smem);
    else if (nt8 == 3) ffn_body<BITS, 3, GATEUP>(p, ex, e, rb, split, row0, nvalid, smem);
    else ffn_body<BITS, 4, GATEUP>(p, ex, e, rb, split, row0, nvalid, smem);
}

template <bool GATEUP>
__global__ void __launch_bounds__(FFN_THREADS, 2) ffn_stream_kernel(const FfnParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    const LayerDev* L = p.L;
    const int e = L->order[blockIdx.y];
    const int tc = blockIdx.x % p.n_tc;
    const int rbs = blockIdx.x / p.n_tc;
    const int rb = rbs / p.ksplit, split = rbs % p.ksplit;
    const int cnt = p.ws.counts[e];
    if (cnt > p.ws.tc_min || tc * CHUNK_TOKENS >= cnt) return;  // larger experts take the tcgen05 path
    const int row0 = p.ws.off_pad[e] + tc * CHUNK_TOKENS;       // physical rows
    const int nvalid = min(CHUNK_TOKENS, cnt - tc * CHUNK_TOKENS);
    const ExpertDev& ex = L->ex[e];
    switch (ex.bits) {
        case 2: ffn_dispatch_tiles<2, GATEUP>(p, ex, e, rb, split, row0, nvalid, smem); break;
        case 3: ffn_dispatch_tiles<3, GATEUP>(p, ex, e, rb, split, row0, nvalid, smem); break;
        case 4: ffn_dispatch_tiles<4, GATEUP>(p, ex, e, rb, split, row0, nvalid, smem); break;
        default: ffn_dispatch_tiles<8, GATEUP>(p, ex, e, rb, split, row0, nvalid, smem); break;
    }
}

template <bool GATEUP>
static cudaError_t launch_one(const FfnParams& p, dim3 grid, cudaStream_t st) {
    cudaError_t err = cudaFuncSetAttribute(ffn_stream_kernel<GATEUP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           p.smem_bytes);
    if (err != cudaSuccess) return err;
    ffn_stream_kernel<GATEUP><<<grid, FFN_THREADS, p.smem_bytes, st>>>(p);
    return cudaGetLastError();
}

// n_tc: 32-token chunks per expert launched; n_rb: weight row blocks; n_experts: experts in L->order.
cudaError_t launch_ffn_stream(const LayerDev* L, const WsDev& ws, int gateup, int n_tc, int n_rb, int ksplit,
                              int n_experts, long long split_stride, int smem_bytes, cudaStream_t st) {
    FfnParams p;
    p.L = L;
    p.ws = ws;
    p.n_tc = n_tc;
    p.ksplit = ksplit;
    p.split_stride = split_stride;
    p.smem_bytes = smem_bytes;
    dim3 grid((unsigned)(n_tc * n_rb * ksplit), (unsigned)n_experts);
    return gateup ? launch_one<true>(p, grid, st) : launch_one<false>(p, grid, st);
}

}  // namespace dyn
