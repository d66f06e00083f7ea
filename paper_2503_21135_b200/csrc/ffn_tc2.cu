// Grouped dequant-GEMM for experts with many tokens (prefill) on PAIRS of SMs: thread-block clusters of two
// CTAs drive one tcgen05.mma.cta_group::2 of M = 256 weight rows x N <= 256 tokens x K = 16.
//
// Why pairs: a tcgen05.mma costs the tensor core at least as long as a 128-token one however few tokens it has,
// and the dequantization of a 256 x 128 weight block costs ~4500 warp instructions however many tokens use
// it.  With M = 256 across two CTAs each CTA dequantizes only ITS 128 rows (8 atoms) per stage, into its own
// tensor memory, for a tile of 256 tokens: half the dequant work per flop of the one-CTA kernel at twice
// the tokens per MMA, so the tensor pipe, not the dequant warps, sets the pace.
//
// Work item of a cluster = (expert, 256-row weight block, tile of <= 256 tokens), K over the whole input axis;
// items are dealt round-robin over the clusters; ring, A buffers, accumulators live across items.
// Per CTA (rank r = 0 leader, 1 peer), 19 warps:
//   warp 16 weights  : bulk copies of the CTA's half block (codes of atoms 8r..8r+7, params of rows 128r..) into a
//                      ring of four small slots; a slot goes back as soon as the stage's warps hold its codes.
//   warp 18 operands : bulk copy of ITS half of the token tile (N/2 tokens: the B operand is split across the
//                      pair) into a ring of four 36 KB slots, freed by the MMAs' commit.  The operand copy is the long
//                      pole of a stage (2000-2800 cycles under load), so it gets the depth; the weights land on
//                      their own barrier and are dequantized while the tile is still in flight.
//   warps 0-15 dequant: a whole atom (16 rows x 128 k) of every OTHER stage each (eight warps per stage): packed
//                      codes -> full fp16 weight (AND-OR, HSUB2, HFMA2 per register pair, the weight s*q+m rounded
//                      once) -> tcgen05.st into the CTA's tensor memory; then wait for the CTA's operand tile and
//                      arrive on the LEADER's a_full barrier (remote arrive for the peer).
//   warp 17 MMA      : in the leader only: waits for both CTAs' A buffers, issues the eight MMAs of the stage
//                      for the pair, commits (multicast) to both CTAs' a_empty / operand-slot / d_full barriers.
//   epilogue         : warps 0-15 of each CTA read their CTA's 128 accumulator rows x N tokens (tcgen05.ld),
//                      SwiGLU -> fp16 h as the down GEMM's operand tiles, or fp32 rows out; then arrive on the
//                      leader's d_empty barrier.
// Tensor memory per CTA: columns 0..255 accumulators (128 rows x 256 tokens), 256..511 four A buffers.
// Every wait is bounded; after an expired wait a CTA leaves its loops and meets its peer at the final
// cluster barrier (the peer's own waits expire within the same bound).
#include <type_traits>

#include "common.cuh"
#include "expand.cuh"
#include "layout.cuh"
#include "tcgen05.cuh"

namespace dyn {

constexpr int T2_DEQ_WARPS = 16;
constexpr int T2_W_PROD = 16, T2_W_MMA = 17, T2_W_PRODX = 18;
constexpr int T2_THREADS = 19 * 32;
constexpr int T2_N = 256;                              // tokens per work item (128 per CTA)
constexpr int T2_WHALF_MAX = 17408;                    // half of the largest packed block (8-bit, G = 64)
constexpr int T2_XTILE = 16 * TC_RG_STRIDE;            // 128 tokens x 128 k: 16 row-group tiles at their buffer pitch
constexpr int T2_POOL_TILES = POOL_GROUP * POOL_TILE_PITCH;       // cached-channel stage: 32 column tiles in a weight slot ...
constexpr int T2_POOL_XG = 16 * 512;                              // ... and their operand tile of 16 row groups in an operand slot
static_assert(T2_POOL_TILES <= T2_WHALF_MAX && T2_POOL_XG <= T2_XTILE, "cached-channel stage does not fit its slots");
// Two rings of four slots.  The operand tiles (36 KB, read by the MMAs; their copy is the long pole of a stage at
// 2000-2800 cycles under load) are freed by the MMAs' commit; the packed weights (read only by the dequant warps, at
// the start of their visit) have small slots that are handed back as soon as the codes are in registers, so the
// weights of a warp's next visit are already there when it comes back.  (Five operand + two weight slots measured
// 2 % slower: the weight wait of ~700 cycles per visit came back.)
constexpr int T2_NW = 4;
constexpr int T2_NX = 4;
constexpr int T2_OFF_PREFIX = 256;                     // item prefix table: MAX_EXPERTS + 1 ints
constexpr int T2_OFF_STAGE = 2048;
constexpr int T2_OFF_XRING = T2_OFF_STAGE + T2_NW * T2_WHALF_MAX;
constexpr int T2_SMEM_BYTES = T2_OFF_XRING + T2_NX * T2_XTILE;
static_assert(T2_OFF_XRING % 1024 == 0 && T2_XTILE % 1024 == 0, "operand slots must stay 1024-byte aligned");
static_assert(T2_OFF_PREFIX + (MAX_EXPERTS + 1) * 4 <= T2_OFF_STAGE, "item table overlaps the stage ring");
static_assert(T2_SMEM_BYTES <= 227 * 1024, "shared memory limit of a CTA");
constexpr uint32_t T2_TMEM_COLS = 512;
constexpr uint32_t T2_COL_A = 256;
constexpr int T2_NA = 4;                               // A buffers of 64 columns: the dequant warps run ahead of the MMA
constexpr int T2_LEAD = 2;                             // stages of the next item dequantized before an item's epilogue

struct T2Params {
    const LayerDev* L;
    WsDev ws;
    int n_rb;       // 256-row weight blocks of this GEMM
    int n_experts;  // experts listed in L->order
};

struct T2Bars {
    uint64_t full[T2_NW], empty[T2_NW];    // per CTA: weight bytes landed / the stage's 8 dequant warps hold the codes
    uint64_t fullx[T2_NX], emptyx[T2_NX];  // per CTA: operand bytes landed / the MMAs that read them are done (commit)
    uint64_t a_full[T2_NA];              // leader only: the 16 dequant warps of the pair that own the stage stored A buffer b
    uint64_t a_empty[T2_NA];                // per CTA: the MMAs that read A buffer b are done (commit)
    uint64_t d_full;                     // per CTA: the item's accumulators are complete (commit)
    uint64_t d_empty;                    // leader only: 32 epilogue warps of the pair have read their accumulators
    uint32_t tmem_base;
    volatile int poison;
};
static_assert(sizeof(T2Bars) <= T2_OFF_PREFIX, "barrier block overlaps the item table");

// One work item of the cluster, as seen by CTA `rank`.
struct T2Item {
    const ExpertDev* ex;
    const uint8_t* wbase;  // first packed block of the item's row block
    int rb, n_valid, n_mma, row0, bits, blk_bytes, n_it;
    int rg_mine0, n_rg_mine;  // this CTA's half of the token tile: first 8-row group and how many hold rows
};

template <bool GATEUP>
__device__ __forceinline__ T2Item t2_decode_item(const T2Params& p, const int* prefix, int g, int& cursor, int n_kc,
                                                 int rank) {
    const LayerDev* L = p.L;
    while (g >= prefix[cursor + 1]) ++cursor;
    const int e = L->order[cursor];
    const int local = g - prefix[cursor];
    const int cnt = p.ws.counts[e];
    const int n_tt = (cnt + T2_N - 1) / T2_N;
    const int tt = local % n_tt;  // tiles of one weight block are neighbours: concurrent clusters share its L2 lines
    T2Item it;
    it.rb = local / n_tt;
    it.n_valid = min(T2_N, cnt - tt * T2_N);
    it.n_mma = (it.n_valid + 31) & ~31;  // N of the pair's MMA; each CTA holds N/2 token rows of B
    it.row0 = p.ws.off_pad[e] + tt * T2_N;
    const int half = it.n_mma >> 1;
    const int nv_mine = max(0, min(half, it.n_valid - rank * half));
    it.n_rg_mine = (nv_mine + 7) >> 3;
    it.rg_mine0 = (it.row0 + rank * half) >> 3;
    it.ex = &L->ex[e];
    it.bits = it.ex->bits;
    it.blk_bytes = it.ex->blk_bytes;
    it.wbase = (GATEUP ? it.ex->w13 : it.ex->w2) + (size_t)it.rb * n_kc * it.blk_bytes;
    const int sig_cnt = (GATEUP && it.ex->switchable) ? L->sig_cnt[e] : 0;
    it.n_it = n_kc + (sig_cnt > 0 ? L->P_pad >> 5 : 0);  // + cached-channel stages of 32 pool columns
    return it;
}

// One (atom, 64-k half) of the CTA's half block -> 32 columns of the A buffer.  a_l: atom within the half
// block (its params are rows 16*a_l .. of the half block's parameter table).
template <int BITS>
__device__ __forceinline__ void t2_dequant_half(const uint8_t* st, uint32_t a_cols, int a_l, int half, int lane, int G,
                                                uint64_t* release) {
    const int gid = lane >> 2;
    const int ngrp = KC / G;
    constexpr int BIAS = BITS == 2 ? 4 : (BITS == 3 ? 3 : ((BITS == 4 || BITS == 6) ? 2 : 0));
    constexpr int NOFF = BITS == 2 ? 5 : (BITS == 3 ? 4 : ((BITS == 4 || BITS == 6) ? 2 : 1));  // distinct offsets 0, step, 2*step, ...
    constexpr int OSTEP = (BITS == 4 || BITS == 6) ? 4 : 2;
    const uint32_t* prm = reinterpret_cast<const uint32_t*>(st + 8 * atom_bytes(BITS));
    const __half2 k1024 = __float2half2_rn(1024.f);
    Codes<BITS> cd;
    load_codes<BITS>(cd, st + a_l * atom_bytes(BITS), lane, half);
    const int g = (G == 64) ? half : 0;
    __half2 S2[2], M2[2][NOFF];
#pragma unroll
    for (int rh = 0; rh < 2; ++rh) {
        const int r = 16 * a_l + gid + 8 * rh;
        const uint32_t pw = prm[r * ngrp + g];
        const __half2 pp = *reinterpret_cast<const __half2*>(&pw);
        S2[rh] = __half2half2(__hmul(__low2half(pp), __ushort_as_half((unsigned short)((15 - BIAS) << 10))));
#pragma unroll
        for (int i = 0; i < NOFF; ++i)  // zero-point times 2^(o - bias), exact
            M2[rh][i] =
                __half2half2(__hmul(__high2half(pp), __ushort_as_half((unsigned short)((15 + OSTEP * i - BIAS) << 10))));
    }
    // codes and parameters are in registers: the weight slot can go back to the producer (second half only)
    if (release) {
        __syncwarp();
        if (lane == 0) mbar_arrive(release);
    }
    uint32_t regs[16];
    auto step = [&](auto S4c) {
        constexpr int S4 = decltype(S4c)::value;
        uint32_t af[4];
        expand<BITS, S4, 0x64006400u>(cd, af);
#pragma unroll
        for (int ri = 0; ri < 4; ++ri) {
            const int oi = code_offset<BITS>(S4, ri >> 1) / OSTEP;
            const __half2 qo = __hsub2(*reinterpret_cast<const __half2*>(&af[ri]), k1024);  // q * 2^o, exact
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
    tc_st_x4(a_cols + 32 * half, regs);
}

template <bool GATEUP>
__global__ void __launch_bounds__(T2_THREADS, 1) ffn_tc2_kernel(const T2Params p) {
    extern __shared__ __align__(1024) uint8_t smem[];
    pdl_prologue();
    const LayerDev* L = p.L;
    const int G = L->G;
    const int K = GATEUP ? L->d : L->f;
    const int n_kc = K / KC;
    const int P_pad = L->P_pad;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;

    T2Bars* B = reinterpret_cast<T2Bars*>(smem);
    int* prefix = reinterpret_cast<int*>(smem + T2_OFF_PREFIX);
    uint8_t* wring = smem + T2_OFF_STAGE;
    uint8_t* xring = smem + T2_OFF_XRING;

    // After an expired wait nothing new starts.  Both CTAs of a pair read the same word (the preceding kernel has
    // completed, and every cluster of this persistent grid starts at launch), so they leave together, before any
    // barrier or tensor memory exists.
    if (*p.ws.status & STATUS_TIMEOUT) return;
    // Item table (identical in both CTAs of the pair): experts above the row threshold contribute
    // (256-token tiles x row blocks) items.
    for (int i = threadIdx.x; i < p.n_experts; i += T2_THREADS) {
        const int cnt = p.ws.counts[L->order[i]];
        prefix[i + 1] = cnt > p.ws.tc_min ? ((cnt + T2_N - 1) / T2_N) * p.n_rb : 0;
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
    // Nothing for this pair: both CTAs see the same table and leave together, before the cluster barrier.
    if (cluster_id >= total) return;

    if (threadIdx.x == 0) {
        for (int i = 0; i < T2_NW; ++i) {
            mbar_init(&B->full[i], 1);
            mbar_init(&B->empty[i], T2_DEQ_WARPS / 2);
        }
        for (int i = 0; i < T2_NX; ++i) {
            mbar_init(&B->fullx[i], 1);
            mbar_init(&B->emptyx[i], 1);
        }
        for (int i = 0; i < T2_NA; ++i) {
            mbar_init(&B->a_full[i], T2_DEQ_WARPS);  // 8 warps of each CTA per stage
            mbar_init(&B->a_empty[i], 1);
        }
        mbar_init(&B->d_full, 1);
        mbar_init(&B->d_empty, 2 * T2_DEQ_WARPS);
        B->poison = 0;
        fence_barrier_init();
    }
    if (warp == T2_W_MMA) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&B->tmem_base)),
                     "r"(T2_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // both CTAs' barriers are initialised before anybody arrives remotely
    tc_fence_after();
    const uint32_t tbase = B->tmem_base;
    volatile int* poison = &B->poison;
    int32_t* status = p.ws.status;
    const uint8_t* xbase = GATEUP ? p.ws.xperm : p.ws.hbuf;
    // Every role walks the same items (static round-robin over the clusters) with its own running stage counter.
    int cursor = 0;
    uint32_t gi = 0;

    if (warp == T2_W_PROD) {
        // ---------------- weight producer (each CTA loads its own half block) ----------------
        bool ok = true;
        for (int g = cluster_id; g < total && ok; g += n_clusters) {
            const T2Item w = t2_decode_item<GATEUP>(p, prefix, g, cursor, n_kc, rank);
            const int code_half = 8 * atom_bytes(w.bits), prm_half = 128 * (KC / G) * 4;
            for (int it = 0; it < w.n_it && ok; ++it, ++gi) {
                const int s = gi % T2_NW, ph = (gi / T2_NW) & 1;
                uint8_t* st = wring + (size_t)s * T2_WHALF_MAX;
                int okl = 1;
                if (lane == 0) okl = mbar_wait_bounded(&B->empty[s], ph ^ 1, poison, status) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, okl, 0) != 0;
                if (!ok) break;
                if (lane == 0) {
                    if (it < n_kc) {
                        const uint8_t* blk = w.wbase + (size_t)it * w.blk_bytes;
                        mbar_arrive_expect_tx(&B->full[s], (uint32_t)(code_half + prm_half));
                        bulk_g2s(st, blk + rank * code_half, (uint32_t)code_half, &B->full[s]);
                        bulk_g2s(st + code_half, blk + block_code_bytes(w.bits) + rank * prm_half, (uint32_t)prm_half,
                                 &B->full[s]);
                    } else {
                        // cached-channel stage: 32 pool columns (whole 256-row tiles: this CTA uses its 128 rows)
                        const int c0 = POOL_GROUP * (it - n_kc);
                        mbar_arrive_expect_tx(&B->full[s], (uint32_t)T2_POOL_TILES);
                        bulk_g2s(st, reinterpret_cast<const uint8_t*>(w.ex->pool_hi) + pool_tile_off(w.rb, c0, P_pad),
                                 (uint32_t)T2_POOL_TILES, &B->full[s]);
                    }
                }
                __syncwarp();
            }
        }
        if (!ok && lane == 0) {
            // let copies in flight land before the CTA's shared memory goes away
            const unsigned long long t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 2000000ull) {
            }
        }
    } else if (warp == T2_W_PRODX) {
        // ---------------- operand producer: this CTA's half of the token tile, one slot per stage ----------------
        bool ok = true;
        for (int g = cluster_id; g < total && ok; g += n_clusters) {
            const T2Item w = t2_decode_item<GATEUP>(p, prefix, g, cursor, n_kc, rank);
            for (int it = 0; it < w.n_it && ok; ++it, ++gi) {
                const int s = gi % T2_NX, ph = (gi / T2_NX) & 1;
                uint8_t* st = xring + (size_t)s * T2_XTILE;
                int okl = 1;
                if (lane == 0) okl = mbar_wait_bounded(&B->emptyx[s], ph ^ 1, poison, status) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, okl, 0) != 0;
                if (!ok) break;
                if (lane == 0) {
                    if (it < n_kc) {
                        mbar_arrive_expect_tx(&B->fullx[s], (uint32_t)(w.n_rg_mine * TC_RG_STRIDE));
                        if (w.n_rg_mine > 0)
                            bulk_g2s(st, xbase + act_off(it, 8 * w.rg_mine0, p.ws.Rcap),
                                     (uint32_t)(w.n_rg_mine * TC_RG_STRIDE), &B->fullx[s]);
                    } else {
                        mbar_arrive_expect_tx(&B->fullx[s], (uint32_t)(w.n_rg_mine * 512));
                        if (w.n_rg_mine > 0)
                            bulk_g2s(st, reinterpret_cast<const uint8_t*>(p.ws.xsig) +
                                             xpool_off(it - n_kc, 8 * w.rg_mine0, p.ws.Rcap),
                                     (uint32_t)(w.n_rg_mine * 512), &B->fullx[s]);
                    }
                }
                __syncwarp();
            }
        }
        if (!ok && lane == 0) {
            const unsigned long long t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 2000000ull) {
            }
        }
    } else if (warp == T2_W_MMA) {
        // ---------------- MMA issuer: leader CTA only, warp-uniform, one elected lane issues ----------------
        if (rank == 0) {
            bool ok = true;
            uint32_t ic = 0;  // items done by this cluster
            auto wait1 = [&](uint64_t* bar, uint32_t par) -> bool {
                int okl = 1;
                if (lane == 0) okl = mbar_wait_bounded_cluster(bar, par, poison, status) ? 1 : 0;
                return __shfl_sync(0xffffffffu, okl, 0) != 0;
            };
            for (int g = cluster_id; g < total && ok; g += n_clusters, ++ic) {
                const T2Item w = t2_decode_item<GATEUP>(p, prefix, g, cursor, n_kc, rank);
                const uint32_t idesc = (1u << 4) | ((uint32_t)(w.n_mma >> 3) << 17) | ((256u >> 4) << 24);
                // the accumulators are free once every epilogue warp of the pair has read the previous item's
                if (ic) ok = wait1(&B->d_empty, (ic - 1) & 1);
                for (int it = 0; it < w.n_it && ok; ++it, ++gi) {
                    const int s = gi % T2_NX;
                    const int b = gi % T2_NA, bph = (gi / T2_NA) & 1;
                    // A buffer b stored by the 16 dequant warps of the pair that own the stage; each also waited for
                    // its CTA's operand tile before it arrived
                    ok = wait1(&B->a_full[b], bph);
                    if (!ok) break;
                    tc_fence_after();
                    const uint8_t* st = xring + (size_t)s * T2_XTILE;
                    const uint32_t a0 = tbase + T2_COL_A + 64 * b;
                    if (it < n_kc) {
                        const uint64_t desc0 = tc_desc(smem_u32(st), 128, TC_RG_STRIDE);
#pragma unroll
                        for (int k8 = 0; k8 < 8; ++k8)
                            tc2_mma_ts_elect(tbase, a0 + 8 * k8, desc0 + (uint64_t)(16 * k8), idesc, (it | k8) ? 1u : 0u);
                    } else {
                        // operand tile of the stage's 32 columns: [row group][k-octet 4][8][8]; step j = two octets
                        const uint32_t xt = smem_u32(st);
                        for (int j = 0; j < 2; ++j)
                            tc2_mma_ts_elect(tbase, a0 + 8 * j, tc_desc(xt + j * 256, 128, 512), idesc, 1u);
                    }
                    tc2_commit_both_elect(&B->a_empty[b]);
                    tc2_commit_both_elect(&B->emptyx[s]);
                }
                if (ok) tc2_commit_both_elect(&B->d_full);
            }
        }
    } else {
        // ---------------- dequant warps, then epilogue ----------------
        // warp -> (TMEM lane quarter q = warp % 4, 16-lane half of it = one atom, stage parity).  A warp's per-stage
        // chain (two barrier waits, shared-memory loads, tensor-memory store and its wait, remote arrive) is
        // latency-bound at well over a thousand cycles however little it computes, so each warp dequantizes a
        // WHOLE atom of every OTHER stage: two stage times per visit.  In the epilogue kh is the token half.
        const int q = warp & 3, asel = (warp >> 2) & 1, kh = warp >> 3;
        const int a_l = 2 * q + asel;        // atom within the CTA's half block
        const int atom_g = 8 * rank + a_l;   // atom within the 256-row block
        const int gid = lane >> 2, tid4 = lane & 3;
        const uint32_t my_lanes = tbase + ((uint32_t)(32 * q + 16 * asel) << 16);
        bool ok = true, clamped = false;
        uint32_t ic = 0;
        // One visit: stage `it` of item w, whose running stage number (ring slots, barrier phases) is gis.
        auto visit = [&](const T2Item& w, int it, uint32_t gis) -> bool {
            const int s = gis % T2_NW, ph = (gis / T2_NW) & 1;     // weight slot (= kh: a warp always uses the same one)
            const int xs = gis % T2_NX, xph = (gis / T2_NX) & 1;   // operand slot
            const int b = gis % T2_NA, bph = (gis / T2_NA) & 1;
            const uint8_t* st = wring + (size_t)s * T2_WHALF_MAX;
            if (!(mbar_wait_bounded(&B->full[s], ph, poison, status) &&
                  mbar_wait_bounded(&B->a_empty[b], bph ^ 1, poison, status)))
                return false;
            tc_fence_after();
            const uint32_t a_cols = my_lanes + T2_COL_A + 64 * b;
            if (it < n_kc) {
                switch (w.bits) {
                    case 2: t2_dequant_half<2>(st, a_cols, a_l, 0, lane, G, nullptr); t2_dequant_half<2>(st, a_cols, a_l, 1, lane, G, &B->empty[s]); break;
                    case 3: t2_dequant_half<3>(st, a_cols, a_l, 0, lane, G, nullptr); t2_dequant_half<3>(st, a_cols, a_l, 1, lane, G, &B->empty[s]); break;
                    case 4: t2_dequant_half<4>(st, a_cols, a_l, 0, lane, G, nullptr); t2_dequant_half<4>(st, a_cols, a_l, 1, lane, G, &B->empty[s]); break;
                    case 6: t2_dequant_half<6>(st, a_cols, a_l, 0, lane, G, nullptr); t2_dequant_half<6>(st, a_cols, a_l, 1, lane, G, &B->empty[s]); break;
                    default: t2_dequant_half<8>(st, a_cols, a_l, 0, lane, G, nullptr); t2_dequant_half<8>(st, a_cols, a_l, 1, lane, G, &B->empty[s]); break;
                }
            } else {
                // cached-channel stage: fp16 tiles [pool column][256 rows] -> A fragments -> tensor memory;
                const int mi = lane >> 3, r = lane & 7;
                for (int j = 0; j < 2; ++j) {
                    uint32_t af[4];
                    const uint32_t addr = smem_u32(st + (j * 16 + (mi >> 1) * 8 + r) * POOL_TILE_PITCH +
                                                   (16 * atom_g + (mi & 1) * 8) * 2);
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(af[0]), "=r"(af[1]), "=r"(af[2]), "=r"(af[3])
                                 : "r"(addr));
                    tc_st_x1(a_cols + 8 * j, af[0], af[2], af[1], af[3]);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&B->empty[s]);  // the tiles are in registers / tensor memory
            }
            tc_wait_st();
            // the arrive below also vouches for this CTA's half of the operand tile (the MMA reads both halves)
            if (!mbar_wait_bounded(&B->fullx[xs], xph, poison, status)) return false;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {  // the barrier lives in the leader: a plain arrive there, a remote one from the peer
                if (rank == 0) mbar_arrive(&B->a_full[b]);
                else mbar_arrive_remote(&B->a_full[b], 0);
            }
            return true;
        };
        // The first T2_LEAD stages of the NEXT item are dequantized before this item's epilogue: their A buffers come
        // free while the last MMAs of this item still run, so when the epilogue hands the accumulators back the MMA
        // warp finds two stages ready instead of waiting for a whole dequantization visit.
        T2Item w = t2_decode_item<GATEUP>(p, prefix, cluster_id, cursor, n_kc, rank);
        int lead_done = 0;                       // stages of w already dequantized (as the previous item's lead)
        for (int g = cluster_id; g < total && ok; g += n_clusters, ++ic) {
            const int bits = w.bits;
            for (int it = lead_done; it < w.n_it && ok; ++it)
                if ((int)((gi + it) & 1) == kh) ok = visit(w, it, gi + it);
            gi += w.n_it;
            T2Item nx = w;
            lead_done = 0;
            if (g + n_clusters < total) {
                nx = t2_decode_item<GATEUP>(p, prefix, g + n_clusters, cursor, n_kc, rank);
                lead_done = nx.n_it < T2_LEAD ? nx.n_it : T2_LEAD;
                for (int it = 0; it < lead_done && ok; ++it)
                    if ((int)((gi + it) & 1) == kh) ok = visit(nx, it, gi + it);
            }
            if (ok) ok = mbar_wait_bounded(&B->d_full, ic & 1, poison, status);
            tc_fence_after();
            if (ok) {
                // this warp: its atom's 16 accumulator rows x the tokens [128*kh, 128*kh + 128) of the tile
                const float scl = __uint_as_float((uint32_t)(127 + x_scale_exp(bits, 8 * atom_g + gid)) << 23);
                // (the next 32 columns are requested before these are processed)
                uint32_t rr[2][16];
                const int ncb = min(4, (w.n_mma - 128 * kh + 31) >> 5);
                if (ncb > 0) tc_ld_x4(my_lanes + 128 * kh, rr[0]);
#pragma unroll
                for (int cb = 0; cb < 4; ++cb) {
                    const int col0 = 128 * kh + 32 * cb;
                    if (cb >= ncb) break;
                    tc_wait_ld();
                    if (cb + 1 < ncb) tc_ld_x4(my_lanes + col0 + 32, rr[(cb + 1) & 1]);
                    const uint32_t (&r)[16] = rr[cb & 1];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if constexpr (GATEUP) {
                            // h of (hidden gid, tokens n0, n0 + 1); lanes gid and gid ^ 1 swap one value each so that
                            // every lane stores one 32-bit pair (hidden gid & ~1, gid | 1) of ONE token
                            const int n0 = col0 + 8 * j + 2 * tid4;
                            float hs[2];
#pragma unroll
                            for (int c = 0; c < 2; ++c) {
                                const float v0 = __uint_as_float(r[4 * j + c]), v1 = __uint_as_float(r[4 * j + 2 + c]);
                                float h = __fdividef(v0, 1.f + __expf(-v0)) * v1;
                                if (n0 + c < w.n_valid) h = clamp_act(h, clamped);   // columns past the last token: ignored
                                h = round_operand(h, p.ws.h_bf16);
                                hs[c] = __half2float(__float2half_rn(h)) * scl;   // exact: scl is a power of two
                            }
                            const int odd = gid & 1;
                            const float give = odd ? hs[0] : hs[1];               // what the partner stores
                            const float got = __shfl_xor_sync(0xffffffffu, give, 4);
                            const int n = n0 + odd;                               // even gid stores token n0, odd gid n0 + 1
                            const __half2 pr = odd ? __floats2half2_rn(got, hs[1]) : __floats2half2_rn(hs[0], got);
                            if (n < w.n_valid) {
                                uint8_t* dst = p.ws.hbuf + act_off(w.rb, (w.row0 + n) & ~7, p.ws.Rcap) + atom_g * 128 +
                                               (n & 7) * 16 + (gid & ~1) * 2;
                                *reinterpret_cast<__half2*>(dst) = pr;
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < 2; ++c) {
                                const int n = col0 + 8 * j + 2 * tid4 + c;
                                if (n < w.n_valid) {
                                    float* yrow = p.ws.ypart + (size_t)(w.row0 + n) * L->d + w.rb * RB + atom_g * 16 + gid;
                                    yrow[0] = __uint_as_float(r[4 * j + c]);
                                    yrow[8] = __uint_as_float(r[4 * j + 2 + c]);
                                }
                            }
                        }
                    }
                }
            }
            // this warp has read its accumulators: hand them back to the leader's MMA warp for the next item
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(&B->d_empty, 0);
            w = nx;
        }
        if (clamped) atomicOr(status, STATUS_RANGE);
    }
    // No CTA of the pair may exit (or free tensor memory) while its peer can still reach it.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == T2_W_MMA) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(T2_TMEM_COLS) : "memory");
    }
}

// Persistent grid: as many CTA pairs as can be resident at once on the current device (pairs must share a TPC; not
// every SM may be pairable), so that the static round-robin over clusters has no second wave.  Also raises the
// kernels' shared-memory limit.  Called once per context at pack time, with the layer's device current.
template <bool GATEUP>
static cudaError_t t2_setup_one(int n_sms, int* clusters_out) {
    cudaError_t err =
        cudaFuncSetAttribute(ffn_tc2_kernel<GATEUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, T2_SMEM_BYTES);
    if (err != cudaSuccess) return err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(n_sms & ~1));
    cfg.blockDim = dim3(T2_THREADS);
    cfg.dynamicSmemBytes = T2_SMEM_BYTES;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int m = 0;
    err = cudaOccupancyMaxActiveClusters(&m, ffn_tc2_kernel<GATEUP>, &cfg);
    if (err != cudaSuccess) return err;
    if (m < 1) return cudaErrorInvalidConfiguration;
    *clusters_out = m < n_sms / 2 ? m : n_sms / 2;
    return cudaSuccess;
}

// clusters_out[0]: down launch, clusters_out[1]: gate/up launch.
cudaError_t setup_ffn_tc2(int n_sms, int* clusters_out) {
    cudaError_t err = t2_setup_one<false>(n_sms, &clusters_out[0]);
    if (err != cudaSuccess) return err;
    return t2_setup_one<true>(n_sms, &clusters_out[1]);
}

// n_rb: 256-row weight blocks; n_experts: experts in L->order; n_clusters: CTA pairs of the persistent grid
// (from setup_ffn_tc2 on this device).
cudaError_t launch_ffn_tc2(const LayerDev* L, const WsDev& ws, int gateup, int n_rb, int n_experts, int n_clusters,
                           cudaStream_t st) {
    T2Params p;
    p.L = L;
    p.ws = ws;
    p.n_rb = n_rb;
    p.n_experts = n_experts;
    if (n_clusters < 1) return cudaErrorInvalidConfiguration;
    return gateup ? launch_pdl_cluster(ffn_tc2_kernel<true>, dim3((unsigned)(2 * n_clusters)), dim3(T2_THREADS),
                                       (size_t)T2_SMEM_BYTES, 2u, st, p)
                  : launch_pdl_cluster(ffn_tc2_kernel<false>, dim3((unsigned)(2 * n_clusters)), dim3(T2_THREADS),
                                       (size_t)T2_SMEM_BYTES, 2u, st, p);
}

}  // namespace dyn
