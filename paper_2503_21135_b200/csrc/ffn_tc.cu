// Grouped dequant-GEMM on the 5th-generation tensor cores for experts with many tokens (prefill).
//
// Persistent grid, one CTA per SM.  One work item = (expert, 256-row weight block = two M=128 tiles, tile
// of <= 128 tokens), K over the whole input axis; items are dealt round-robin and the ring, the A buffers
// and tensor memory live across items.  Roles (18 warps):
//   warp 16 producer : bulk async copies of the packed block and of the activation operand tile
//                      (8-row groups, K-major no-swizzle core matrices) into a 3-stage ring.
//   warps 0-15 dequant: one 16-row atom each; expand packed codes in registers and store the dequantized
//                      fp16 weights with
//                      tcgen05.st.16x256b straight into TENSOR MEMORY as the A operand: the packed
//                      fragment layout (layout.cuh) is exactly that instruction's register layout, so
//                      dequantized weights never touch shared memory.  Per register pair: one AND-OR
//                      (1024 + q*2^o in place), one HSUB2 (exact q*2^o), one HFMA2
//                      ((q*2^o) * (s*2^-bias) + m*2^(o-bias)): the weight s*q + m rounded ONCE to fp16,
//                      times the power of two that the pre-scaled activations undo.
//   warp 17 MMA      : one thread issues tcgen05.mma.kind::f16 (A from TMEM, B from shared memory,
//                      fp32 accumulators in TMEM); tcgen05.commit releases ring slots and A buffers.
// Gate/up: the significant-channel correction follows as extra 16-channel stages (fp16 tiles of the
// active cached channels through ldmatrix -> tcgen05.st); epilogue = tcgen05.ld, SwiGLU, fp16 h written
// as the down GEMM's operand tiles (pre-scaled).  Down: fp32 rows out.
// TMEM: columns 0..255 accumulators (two M tiles x 128 tokens), 256..511 two A buffers.
#include <type_traits>

#include "common.cuh"
#include "expand.cuh"
#include "layout.cuh"
#include "tcgen05.cuh"

namespace dyn {

constexpr int TC_DEQ_WARPS = 16;                    // one 16-row atom each: enough warps to hide the dequant latency
constexpr int TC_APW = 1;                           // atoms per dequant warp
constexpr int TC_THREADS = (TC_DEQ_WARPS + 2) * 32;
constexpr int TC_N = 128;
constexpr int TC_WBLK_MAX = 34816;                  // largest packed block (8-bit, G = 64)
constexpr int TC_XTILE = 16 * TC_RG_STRIDE;         // 128 tokens x 128 k fp16: 16 row-group tiles at their buffer pitch
constexpr int TC_STAGE_BYTES = TC_WBLK_MAX + TC_XTILE;
constexpr int TC_OFF_PREFIX = 256;                  // item prefix table: MAX_EXPERTS + 1 ints
constexpr int TC_OFF_STAGE = 2048;
static_assert(TC_OFF_PREFIX + (MAX_EXPERTS + 1) * 4 <= TC_OFF_STAGE, "item table overlaps the stage ring");
constexpr int TC_NS = 3;                            // ring depth: must cover the L2 latency of the operand tiles
constexpr int TC_SMEM_BYTES = TC_OFF_STAGE + TC_NS * TC_STAGE_BYTES;
constexpr int TC_SIG_TILE_STRIDE = 528;
constexpr uint32_t TC_TMEM_COLS = 512;
constexpr uint32_t TC_COL_A = 256;

struct TcParams {
    const LayerDev* L;
    WsDev ws;
    int n_rb;       // 256-row weight blocks of this GEMM
    int n_experts;  // experts listed in L->order
};

struct TcBars {
    uint64_t full[TC_NS], empty[TC_NS], a_full[2], a_empty[2], d_full, d_empty;
    uint32_t tmem_base;
    volatile int poison;
};

// Dequantize one packed block stage into the A buffer: this warp's two atoms, eight MMA steps.
template <int BITS>
__device__ __forceinline__ void tc_dequant_stage(const uint8_t* st, uint32_t a_lanes, int atom0, int lane, int G) {
    const int gid = lane >> 2;
    const int ngrp = KC / G;
    constexpr int BIAS = BITS == 2 ? 4 : (BITS == 3 ? 3 : (BITS == 4 ? 2 : 0));
    constexpr int NOFF = BITS == 2 ? 5 : (BITS == 3 ? 4 : (BITS == 4 ? 2 : 1));   // distinct offsets 0, step, 2*step, ...
    constexpr int OSTEP = BITS == 4 ? 4 : 2;
    const uint32_t* prm = reinterpret_cast<const uint32_t*>(st + block_code_bytes(BITS));
    const __half2 k1024 = __float2half2_rn(1024.f);
#pragma unroll
    for (int a = 0; a < TC_APW; ++a) {
        const int atom = atom0 + a;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            Codes<BITS> cd;
            load_codes<BITS>(cd, st + atom * atom_bytes(BITS), lane, half);
            const int g = (G == 64) ? half : 0;
            __half2 S2[2], M2[2][NOFF];
#pragma unroll
            for (int rh = 0; rh < 2; ++rh) {
                const int r = 16 * atom + gid + 8 * rh;
                const uint32_t pw = prm[r * ngrp + g];
                const __half2 pp = *reinterpret_cast<const __half2*>(&pw);
                S2[rh] = __half2half2(__hmul(__low2half(pp), __ushort_as_half((unsigned short)((15 - BIAS) << 10))));
#pragma unroll
                for (int i = 0; i < NOFF; ++i)  // zero-point times 2^(o - bias), exact
                    M2[rh][i] = __half2half2(
                        __hmul(__high2half(pp), __ushort_as_half((unsigned short)((15 + OSTEP * i - BIAS) << 10))));
            }
            uint32_t regs[16];
            auto step = [&](auto S4c) {
                constexpr int S4 = decltype(S4c)::value;
                uint32_t af[4];
                expand<BITS, S4, 0x64006400u>(cd, af);
#pragma unroll
                for (int ri = 0; ri < 4; ++ri) {
                    const int oi = code_offset<BITS>(S4, ri >> 1) / OSTEP;
                    const __half2 qo = __hsub2(*reinterpret_cast<const __half2*>(&af[ri]), k1024);   // q * 2^o, exact
                    const __half2 v = __hfma2(qo, S2[ri & 1], M2[ri & 1][oi]);
                    af[ri] = *reinterpret_cast<const uint32_t*>(&v);
                }
                // fragment (rowhalf, h) -> TMEM register order of the 16x256b shape: (row, col pair)
                regs[4 * S4 + 0] = af[0];
                regs[4 * S4 + 1] = af[2];
                regs[4 * S4 + 2] = af[1];
                regs[4 * S4 + 3] = af[3];
            };
            step(std::integral_constant<int, 0>{});
            step(std::integral_constant<int, 1>{});
            step(std::integral_constant<int, 2>{});
            step(std::integral_constant<int, 3>{});
            tc_st_x4(a_lanes + ((uint32_t)(16 * a) << 16) + 32 * half, regs);
        }
    }
}

// One work item = (expert, 256-row weight block, tile of <= 128 tokens).
struct TcItem {
    const ExpertDev* ex;
    const uint8_t* wbase;  // first packed block of the item's row block
    int rb, n_valid, n_rg, n_mma, row0, rg0, bits, blk_bytes, n_it;
};

// Item g of the launch: experts in L->order, items of one expert numbered [row block][token tile].  The
// cursor only moves forward (a CTA's items ascend), so the search is a few steps per item.
template <bool GATEUP>
__device__ __forceinline__ TcItem tc_decode_item(const TcParams& p, const int* prefix, int g, int& cursor, int n_kc) {
    const LayerDev* L = p.L;
    while (g >= prefix[cursor + 1]) ++cursor;
    const int e = L->order[cursor];
    const int local = g - prefix[cursor];
    const int cnt = p.ws.counts[e];
    const int n_tt = (cnt + TC_N - 1) / TC_N;
    const int tt = local % n_tt;
    TcItem it;
    it.rb = local / n_tt;
    it.n_valid = min(TC_N, cnt - tt * TC_N);
    it.n_rg = (it.n_valid + 7) >> 3;
    it.n_mma = (it.n_valid + 15) & ~15;
    it.row0 = p.ws.off_pad[e] + tt * TC_N;
    it.rg0 = it.row0 >> 3;
    it.ex = &L->ex[e];
    it.bits = it.ex->bits;
    it.blk_bytes = it.ex->blk_bytes;
    it.wbase = (GATEUP ? it.ex->w13 : it.ex->w2) + (size_t)it.rb * n_kc * it.blk_bytes;
    const int sig_cnt = (GATEUP && it.ex->switchable) ? L->sig_cnt[e] : 0;
    it.n_it = n_kc + (sig_cnt > 0 ? (L->P_pad + 63) >> 6 : 0);  // + cached-channel stages of 64 pool columns
    return it;
}

template <bool GATEUP>
__global__ void __launch_bounds__(TC_THREADS, 1) ffn_tc_kernel(const TcParams p) {
    extern __shared__ __align__(1024) uint8_t smem[];
    pdl_prologue();
    const LayerDev* L = p.L;
    const int G = L->G;
    const int K = GATEUP ? L->d : L->f;
    const int n_kc = K / KC;
    const int P_pad = L->P_pad;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    TcBars* B = reinterpret_cast<TcBars*>(smem);
    int* prefix = reinterpret_cast<int*>(smem + TC_OFF_PREFIX);
    uint8_t* stages = smem + TC_OFF_STAGE;

    // Item table: experts above the row threshold contribute (token tiles x row blocks) items.
    for (int i = threadIdx.x; i < p.n_experts; i += TC_THREADS) {
        const int cnt = p.ws.counts[L->order[i]];
        prefix[i + 1] = cnt > p.ws.tc_min ? ((cnt + TC_N - 1) / TC_N) * p.n_rb : 0;
    }
    __syncthreads();
    if (warp == 0) {
        int run = 0;
        for (int i0 = 0; i0 < p.n_experts; i0 += 32) {
            const int i = i0 + lane;
            int v = i < p.n_experts ? prefix[i + 1] : 0;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, v, d);
                if (lane >= d) v += u;
            }
            if (i < p.n_experts) prefix[i + 1] = run + v;
            run += __shfl_sync(0xffffffffu, v, 31);
        }
        if (lane == 0) prefix[0] = 0;
    }
    __syncthreads();
    const int total = prefix[p.n_experts];
    // Nothing to do (no expert above the threshold), or an earlier wait expired: leave before any
    // tensor memory is allocated.
    if ((int)blockIdx.x >= total || *p.ws.status != STATUS_OK) return;

    if (threadIdx.x == 0) {
        for (int i = 0; i < TC_NS; ++i) {
            mbar_init(&B->full[i], 1);
            mbar_init(&B->empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&B->a_full[i], TC_DEQ_WARPS);
            mbar_init(&B->a_empty[i], 1);
        }
        mbar_init(&B->d_full, 1);
        mbar_init(&B->d_empty, TC_DEQ_WARPS);
        B->poison = 0;
        fence_barrier_init();
    }
    if (warp == TC_DEQ_WARPS + 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&B->tmem_base)),
                     "r"(TC_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = B->tmem_base;
    volatile int* poison = &B->poison;
    int32_t* status = p.ws.status;
    const uint8_t* xbase = GATEUP ? p.ws.xperm : p.ws.hbuf;
    // Every role walks the same items (static round-robin over the persistent grid) and keeps its own
    // running stage counter gi: ring slots and A buffers carry their phases across items, so the
    // producer prefetches the next item's first stages while this item's epilogue runs.
    int cursor = 0;
    uint32_t gi = 0;

    if (warp == TC_DEQ_WARPS) {
        // ---------------- producer ----------------
        bool ok = true;
        for (int g = blockIdx.x; g < total && ok; g += gridDim.x) {
            const TcItem w = tc_decode_item<GATEUP>(p, prefix, g, cursor, n_kc);
            for (int it = 0; it < w.n_it && ok; ++it, ++gi) {
                const int s = gi % TC_NS, ph = (gi / TC_NS) & 1;  // shared-memory ring slot
                uint8_t* st = stages + (size_t)s * TC_STAGE_BYTES;
                int okl = 1;
                if (lane == 0) okl = mbar_wait_bounded(&B->empty[s], ph ^ 1, poison, status) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, okl, 0) != 0;
                if (!ok) break;
                if (it < n_kc) {
                    if (lane == 0) {
                        // two copies per stage: the packed block and the operand tile (chunk-major: contiguous)
                        mbar_arrive_expect_tx(&B->full[s], (uint32_t)(w.blk_bytes + w.n_rg * TC_RG_STRIDE));
                        bulk_g2s(st, w.wbase + (size_t)it * w.blk_bytes, (uint32_t)w.blk_bytes, &B->full[s]);
                        bulk_g2s(st + TC_WBLK_MAX, xbase + act_off(it, 8 * w.rg0, p.ws.Rcap),
                                 (uint32_t)(w.n_rg * TC_RG_STRIDE), &B->full[s]);
                    }
                } else if (lane == 0) {
                    // cached-channel stage: up to 64 pool columns = one tile copy + one operand copy per 32 columns
                    const int c0 = 64 * (it - n_kc), ngr = min(2, (P_pad - c0) >> 5);
                    mbar_arrive_expect_tx(&B->full[s],
                                          (uint32_t)(ngr * POOL_GROUP * POOL_TILE_PITCH + ngr * w.n_rg * 512));
                    bulk_g2s(st, reinterpret_cast<const uint8_t*>(w.ex->pool_hi) + pool_tile_off(w.rb, c0, P_pad),
                             (uint32_t)(ngr * POOL_GROUP * POOL_TILE_PITCH), &B->full[s]);
                    for (int j = 0; j < ngr; ++j)
                        bulk_g2s(st + TC_WBLK_MAX + j * 8192,
                                 reinterpret_cast<const uint8_t*>(p.ws.xsig) +
                                     xpool_off((c0 >> 5) + j, 8 * w.rg0, p.ws.Rcap),
                                 (uint32_t)(w.n_rg * 512), &B->full[s]);
                }
                __syncwarp();
            }
        }
        if (!ok && lane == 0) {
            const unsigned long long t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 2000000ull) {
            }
        }
    } else if (warp == TC_DEQ_WARPS + 1) {
        // ---------------- MMA issuer (one thread) ----------------
        if (lane == 0) {
            bool ok = true;
            uint32_t ic = 0;  // items done by this CTA
            for (int g = blockIdx.x; g < total && ok; g += gridDim.x, ++ic) {
                const TcItem w = tc_decode_item<GATEUP>(p, prefix, g, cursor, n_kc);
                const uint32_t idesc = (1u << 4) | ((uint32_t)(w.n_mma >> 3) << 17) | (8u << 24);
                // the accumulators are free once every epilogue warp has read the previous item's out
                if (ic) ok = mbar_wait_bounded(&B->d_empty, (ic - 1) & 1, poison, status);
                for (int it = 0; it < w.n_it && ok; ++it, ++gi) {
                    const int s = gi % TC_NS, ph = (gi / TC_NS) & 1;  // shared-memory ring slot
                    const int b = gi & 1, bph = (gi >> 1) & 1;        // tensor-memory A buffer
                    const uint8_t* st = stages + (size_t)s * TC_STAGE_BYTES;
                    ok = mbar_wait_bounded(&B->full[s], ph, poison, status) &&
                         mbar_wait_bounded(&B->a_full[b], bph, poison, status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t xt = smem_u32(st + TC_WBLK_MAX);
                    if (it < n_kc) {
                        // One thread feeds the tensor core: keep the per-instruction work to a few integer adds
                        // (the descriptor of MMA step k8 is the stage's descriptor plus k8 * 256 B >> 4).
                        const uint64_t desc0 = tc_desc(xt, 128, TC_RG_STRIDE);
                        const uint32_t a0 = tbase + TC_COL_A + 128 * b;
                        const uint32_t first = it ? 1u : 0u;
#pragma unroll
                        for (int k8 = 0; k8 < 8; ++k8) {
                            tc_mma_ts(tbase, a0 + 8 * k8, desc0 + (uint64_t)(16 * k8), idesc, k8 ? 1u : first);
                            tc_mma_ts(tbase + 128, a0 + 64 + 8 * k8, desc0 + (uint64_t)(16 * k8), idesc,
                                      k8 ? 1u : first);
                        }
                    } else {
                        const int nsub = min(4, (P_pad - 64 * (it - n_kc)) >> 4);  // 16-column MMA steps in this stage
                        const uint32_t a0 = tbase + TC_COL_A + 128 * b;
                        for (int j = 0; j < nsub; ++j) {
                            // operand tile of the 32-column group j/2: [row group][k-octet 4][8][8]; step (j & 1)
                            // = two octets
                            const uint64_t dsc = tc_desc(xt + (j >> 1) * 8192 + (j & 1) * 256, 128, 512);
                            tc_mma_ts(tbase, a0 + 8 * j, dsc, idesc, 1u);
                            tc_mma_ts(tbase + 128, a0 + 64 + 8 * j, dsc, idesc, 1u);
                        }
                    }
                    tc_commit(&B->a_empty[b]);
                    tc_commit(&B->empty[s]);
                }
                if (ok) tc_commit(&B->d_full);
            }
        }
    } else {
        // ---------------- dequant warps, then epilogue ----------------
        // warp -> (TMEM lane quarter q = warp % 4, M tile, which 16-lane half of the quarter)
        const int q = warp & 3, mt = (warp >> 2) & 1, asel = warp >> 3;
        const int atom0 = 8 * mt + 2 * q + asel;
        const int gid = lane >> 2, tid4 = lane & 3;
        const uint32_t my_lanes = tbase + ((uint32_t)(32 * q + 16 * asel) << 16);
        bool ok = true;
        uint32_t ic = 0;  // items done by this CTA
        for (int g = blockIdx.x; g < total && ok; g += gridDim.x, ++ic) {
        const TcItem w = tc_decode_item<GATEUP>(p, prefix, g, cursor, n_kc);
        const int bits = w.bits, n_valid = w.n_valid, n_mma = w.n_mma, rb = w.rb, rg0 = w.rg0, row0 = w.row0;
        for (int it = 0; it < w.n_it && ok; ++it, ++gi) {
            const int s = gi % TC_NS, ph = (gi / TC_NS) & 1;  // shared-memory ring slot
            const int b = gi & 1, bph = (gi >> 1) & 1;        // tensor-memory A buffer
            const uint8_t* st = stages + (size_t)s * TC_STAGE_BYTES;
            ok = mbar_wait_bounded(&B->full[s], ph, poison, status) &&
                 mbar_wait_bounded(&B->a_empty[b], bph ^ 1, poison, status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_lanes = my_lanes + TC_COL_A + 128 * b + 64 * mt;
            if (it < n_kc) {
                switch (bits) {
                    case 2: tc_dequant_stage<2>(st, a_lanes, atom0, lane, G); break;
                    case 3: tc_dequant_stage<3>(st, a_lanes, atom0, lane, G); break;
                    case 4: tc_dequant_stage<4>(st, a_lanes, atom0, lane, G); break;
                    default: tc_dequant_stage<8>(st, a_lanes, atom0, lane, G); break;
                }
            } else {
                // significant-channel stage: fp16 tiles [slot][256 rows] -> A fragments -> TMEM
                const int mi = lane >> 3, r = lane & 7;
                const int nsub = min(4, (P_pad - 64 * (it - n_kc)) >> 4);
                for (int j = 0; j < nsub; ++j) {
#pragma unroll
                    for (int a = 0; a < TC_APW; ++a) {
                        uint32_t af[4];
                        const uint32_t addr = smem_u32(st + (j * 16 + (mi >> 1) * 8 + r) * TC_SIG_TILE_STRIDE +
                                                       (16 * (atom0 + a) + (mi & 1) * 8) * 2);
                        asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                                     : "=r"(af[0]), "=r"(af[1]), "=r"(af[2]), "=r"(af[3])
                                     : "r"(addr));
                        tc_st_x1(a_lanes + ((uint32_t)(16 * a) << 16) + 8 * j, af[0], af[2], af[1], af[3]);
                    }
                }
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&B->a_full[b]);
        }
        if (ok) ok = mbar_wait_bounded(&B->d_full, ic & 1, poison, status);
        tc_fence_after();
        if (ok) {
            const float scl[2] = {__uint_as_float((uint32_t)(127 + x_scale_exp(bits, 8 * atom0 + gid)) << 23),
                                  __uint_as_float((uint32_t)(127 + x_scale_exp(bits, 8 * (atom0 + 1) + gid)) << 23)};
#pragma unroll
            for (int a = 0; a < TC_APW; ++a) {
                const int atom = atom0 + a;
                for (int cb = 0; cb * 32 < n_mma; ++cb) {
                    uint32_t r[16];
                    tc_ld_x4(my_lanes + ((uint32_t)(16 * a) << 16) + 128 * mt + 32 * cb, r);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            const int n = 32 * cb + 8 * j + 2 * tid4 + c;
                            const float v0 = __uint_as_float(r[4 * j + c]), v1 = __uint_as_float(r[4 * j + 2 + c]);
                            if (n < n_valid) {
                                if constexpr (GATEUP) {
                                    const float h = v0 / (1.f + expf(-v0)) * v1;
                                    const float h16 = __half2float(__float2half_rn(h));
                                    uint8_t* dst = p.ws.hbuf + act_off(rb, 8 * (rg0 + (n >> 3)), p.ws.Rcap) +
                                                   atom * 128 + (n & 7) * 16 + gid * 2;
                                    *reinterpret_cast<__half*>(dst) = __float2half_rn(h16 * scl[a]);
                                } else {
                                    float* yrow = p.ws.ypart + (size_t)(row0 + n) * L->d + rb * RB + atom * 16 + gid;
                                    yrow[0] = v0;
                                    yrow[8] = v1;
                                }
                            }
                        }
                    }
                }
            }
        }
        // this warp has read its accumulators: hand them back to the MMA warp for the next item
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&B->d_empty);
        }  // items
    }
    tc_fence_before();
    __syncthreads();
    if (warp == TC_DEQ_WARPS + 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(TC_TMEM_COLS) : "memory");
    }
}

template <bool GATEUP>
static cudaError_t launch_tc_one(const TcParams& p, dim3 grid, cudaStream_t st) {
    cudaError_t err =
        cudaFuncSetAttribute(ffn_tc_kernel<GATEUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES);
    if (err != cudaSuccess) return err;
    return launch_pdl(ffn_tc_kernel<GATEUP>, grid, dim3(TC_THREADS), (size_t)TC_SMEM_BYTES, st, p);
}

// n_rb: 256-row weight blocks; n_experts: experts in L->order; n_sms: one persistent CTA per SM.
cudaError_t launch_ffn_tc(const LayerDev* L, const WsDev& ws, int gateup, int n_rb, int n_experts, int n_sms,
                          cudaStream_t st) {
    TcParams p;
    p.L = L;
    p.ws = ws;
    p.n_rb = n_rb;
    p.n_experts = n_experts;
    dim3 grid((unsigned)n_sms);
    return gateup ? launch_tc_one<true>(p, grid, st) : launch_tc_one<false>(p, grid, st);
}

}  // namespace dyn
