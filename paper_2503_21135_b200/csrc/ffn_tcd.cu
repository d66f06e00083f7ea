// Decode-sized grouped dequant-GEMM on the 5th-generation tensor cores: experts with few tokens, where
// the forward is bound by streaming the packed weights from HBM and every instruction per weight counts.
//
// Persistent grid, one CTA per SM, 19 warps.  Work item = (expert, 256-row weight block = two M=128
// tiles, chunk of <= 32 tokens, K split); items are dealt round-robin, the stage ring, the tensor-memory
// buffers and all barrier phases live across items.
//   warp 0     producer : one bulk copy of the packed block and one of the operand tile per stage into a
//                         byte-granular ring (16 slots); also prepares the stage's MMA operand descriptor.
//   warps 1-2  MMA      : one M tile each; warp-uniform code, one elected lane issues tcgen05.mma.kind::f16
//                         (A in tensor memory, B = operand tile in shared memory) into a FRESH accumulator
//                         buffer per quantization group and commits it.
//   warps 3-10 expand   : two 16-row atoms each.  Codes are used IN PLACE: a field masked where it sits is the
//                         fp16 subnormal q * 2^(o-24), so ONE logical instruction per register pair turns
//                         packed words into A-operand registers, stored with tcgen05.st.16x256b straight into
//                         tensor memory (the packed fragment order is that instruction's register layout).
//                         The activations carry 2^(bias-o(k)) (gather kernel), so a group's dot product is
//                         2^(bias-24) * sum_k q_k x_k exactly.
//   warps 11-18 fold    : read each group's accumulators back (tcgen05.ld) and fold them into fp32 registers:
//                         total += (s * 2^(24-bias)) * acc + m * sum_k x_k  (scale and zero enter once per
//                         group and row, not once per weight), then release the stage; epilogue.
// Measured on B200 this kernel is slower than the streaming kernel (445 vs 278 us per forward at 64 tokens of
// the decode shape): a tcgen05.mma costs its issuing warp ~50 cycles whatever N is, and the per-stage
// expand -> MMA -> fold chain (about 1000 cycles per role) is not hidden by two A and two accumulator buffers.
// It is kept selectable (dynamo_set_decode_kernel) and tested; the streaming kernel is the default.
// Gate/up: cached-channel stages (fp16 tiles of the whole pool x activations that are zero for channels
// not significant now) add straight into the totals; epilogue SwiGLU -> fp16 h written as the down GEMM's
// operand tiles with their half-chunk sums.  Down: fp32 rows per K split.
// Tensor memory: columns 0..127 two accumulator buffers (two M tiles x 32 tokens each), 128..383 two A buffers.
#include <type_traits>

#include "common.cuh"
#include "expand.cuh"
#include "layout.cuh"
#include "tcgen05.cuh"

namespace dyn {

constexpr int TD_EXP_WARPS = 8;                          // code expansion -> tensor memory, two atoms each
constexpr int TD_FOLD_WARPS = 8;                         // accumulator groups -> fp32 totals, epilogue

// Warp roles.  The producer and the MMA issuers take the LOWEST warp ids: they issue few instructions but every
// one is on the critical path, and the schedulers favour older (lower) warps.
constexpr int TD_MMA_WARPS = 2;   // 2: one per M tile; 4: (M tile) x (stage parity)
constexpr int TD_W_PROD = 0, TD_W_MMA = 1, TD_W_EXP = TD_W_MMA + TD_MMA_WARPS, TD_W_FOLD = TD_W_EXP + TD_EXP_WARPS;
constexpr int TD_THREADS = (TD_W_FOLD + TD_FOLD_WARPS) * 32;
constexpr int TD_N = 32;                                 // tokens per work item
constexpr int TD_NS = 16;                                // queue slots of the byte-granular stage ring
constexpr int TD_OFF_PREFIX = 640;                       // item prefix table: MAX_EXPERTS + 1 ints
constexpr int TD_OFF_PART = 2048;                        // partial h sums [2][16 atoms][32 tokens] fp32
constexpr int TD_OFF_STAGE = TD_OFF_PART + 2 * 16 * TD_N * 4;
constexpr int TD_SMEM_BYTES = 227 * 1024;
// Stage ring: a stage takes only the bytes it needs (a 2-bit block is 9 KB, an 8-bit one 34 KB), so low-bit
// experts keep ~15 stages in flight: the bytes in flight per SM, not the stage count, must cover HBM latency.
constexpr int TD_RING_BYTES = (TD_SMEM_BYTES - TD_OFF_STAGE) & ~127;
constexpr int TD_SIG_TILE_STRIDE = POOL_TILE_PITCH;
constexpr int TD_SUM_OFF = TC_TILE_BYTES;                // per 8-row group tile: [half chunk 2][row 8] fp32 sums
constexpr uint32_t TD_TMEM_COLS = 512;
constexpr uint32_t TD_COL_A = 128;
// High word of the K-major no-swizzle operand descriptor: SBO >> 4 (stride between 8-row groups) | version bit 46.
constexpr uint32_t TD_DESC_HI_W = (TC_RG_STRIDE >> 4) | (1u << 14);   // activation tiles at their buffer pitch
constexpr uint32_t TD_DESC_HI_P = (512u >> 4) | (1u << 14);            // cached-channel operand tiles
static_assert(TD_OFF_PREFIX + (MAX_EXPERTS + 1) * 4 <= TD_OFF_PART, "item table overlaps the partial sums");
static_assert(TD_SMEM_BYTES <= 227 * 1024, "shared memory budget");

// Operand tile offset inside a stage: after the packed block / after the cached-channel tiles.
__device__ __forceinline__ int td_xoff_weight(int blk_bytes) { return (blk_bytes + 127) & ~127; }
__device__ __forceinline__ int td_xoff_pool(int ngr) { return ngr * POOL_GROUP * POOL_TILE_PITCH; }

struct TdParams {
    const LayerDev* L;
    WsDev ws;
    int n_rb;       // 256-row weight blocks of this GEMM
    int n_experts;  // experts listed in L->order
    int ksplit;     // K splits (down GEMM at small token counts)
    long long split_stride;  // floats between the partial outputs of two K splits
};

struct TdBars {
    uint64_t full[TD_NS], empty[TD_NS], a_full[2], a_empty[2], d_full[2], d_empty[2], epi;
    int off[TD_NS];   // ring offset of the stage in queue slot q (written by the producer before it arrives)
    uint32_t xdesc[TD_NS];  // low word of the stage's operand-tile MMA descriptor (address >> 4 | LBO)
    int size[TD_NS];  // bytes the stage holds in the ring (producer only)
    uint32_t tmem_base;
    volatile int poison;
};

static_assert(sizeof(TdBars) <= TD_OFF_PREFIX, "barrier block overlaps the item table");

// One work item.
struct TdItem {
    const ExpertDev* ex;
    const uint8_t* wbase;  // first packed block of the item's row block
    int rb, split, n_valid, n_rg, n_mma, row0, rg0, bits, blk_bytes, kc0, n_w, n_ps;
};

// Item g of the launch: experts in L->order; items of one expert numbered [row block][K split][token chunk]
// (chunks of one weight block are neighbours: they share L2 lines).
template <bool GATEUP>
__device__ __forceinline__ TdItem td_decode_item(const TdParams& p, const int* prefix, int g, int& cursor, int n_kc) {
    const LayerDev* L = p.L;
    while (g >= prefix[cursor + 1]) ++cursor;
    const int e = L->order[cursor];
    const int local = g - prefix[cursor];
    const int cnt = p.ws.counts[e];
    const int n_ch = (cnt + TD_N - 1) / TD_N;
    const int ch = local % n_ch, rbs = local / n_ch;
    TdItem it;
    it.rb = rbs / p.ksplit;
    it.split = rbs % p.ksplit;
    it.n_valid = min(TD_N, cnt - ch * TD_N);
    it.n_rg = (it.n_valid + 7) >> 3;
    it.n_mma = (it.n_valid + 15) & ~15;
    it.row0 = p.ws.off_pad[e] + ch * TD_N;
    it.rg0 = it.row0 >> 3;
    it.ex = &L->ex[e];
    it.bits = it.ex->bits;
    it.blk_bytes = it.ex->blk_bytes;
    it.wbase = (GATEUP ? it.ex->w13 : it.ex->w2) + (size_t)it.rb * n_kc * it.blk_bytes;
    it.kc0 = (int)(((long long)it.split * n_kc) / p.ksplit);
    it.n_w = (int)(((long long)(it.split + 1) * n_kc) / p.ksplit) - it.kc0;
    const int sig_cnt = (GATEUP && it.ex->switchable) ? L->sig_cnt[e] : 0;
    it.n_ps = sig_cnt > 0 ? (L->P_pad + 63) >> 6 : 0;  // cached-channel stages of 64 pool columns
    return it;
}

// Packed block stage -> A buffer: this warp's atom, eight MMA steps, one logical op per register pair.
template <int BITS>
__device__ __forceinline__ void td_expand_stage(const uint8_t* st, uint32_t a_lanes, int atom, int lane) {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        Codes<BITS> cd;
        load_codes<BITS>(cd, st + atom * atom_bytes(BITS), lane, half);
        uint32_t regs[16];
        auto step = [&](auto S4c) {
            constexpr int S4 = decltype(S4c)::value;
            uint32_t af[4];
            expand<BITS, S4, 0u>(cd, af);
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
        tc_st_x4(a_lanes + 32 * half, regs);
    }
}

// Expand warps (0..7): TMEM lane quarter q = warp % 4, M tile = warp / 4, both 16-lane halves = two atoms.
// One item: for every stage wait for the data and for a free A buffer, expand, publish the buffer.
template <bool GATEUP>
__device__ __forceinline__ bool td_expand_item(const TdParams& p, const TdItem& w, TdBars* B, uint8_t* stages,
                                               uint32_t tbase, uint32_t& gi, volatile int* poison) {
    int32_t* status = p.ws.status;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q = warp & 3, mt = (warp - TD_W_EXP) >> 2;  // a warp reaches the TMEM lane quarter warp % 4
    const int atom0 = 8 * mt + 2 * q;
    const uint32_t my_lanes = tbase + ((uint32_t)(32 * q) << 16);
    const int P_pad = p.L->P_pad;
    const int bits = w.bits;
    const int n_it = w.n_w + w.n_ps;
    for (int it = 0; it < n_it; ++it, ++gi) {
        const int s = gi % TD_NS, ph = (gi / TD_NS) & 1;  // shared-memory ring slot
        const int b = gi & 1, bph = (gi >> 1) & 1;        // tensor-memory A buffer
        if (!(mbar_wait_bounded(&B->full[s], ph, poison, status) &&
              mbar_wait_bounded(&B->a_empty[b], bph ^ 1, poison, status)))
            return false;
        tc_fence_after();
        const uint8_t* st = stages + B->off[s];
        const uint32_t a_lanes = my_lanes + TD_COL_A + 128 * b + 64 * mt;
        if (it < w.n_w) {
#pragma unroll
            for (int a = 0; a < 2; ++a) {
                const uint32_t al = a_lanes + ((uint32_t)(16 * a) << 16);
                switch (bits) {
                    case 2: td_expand_stage<2>(st, al, atom0 + a, lane); break;
                    case 3: td_expand_stage<3>(st, al, atom0 + a, lane); break;
                    case 4: td_expand_stage<4>(st, al, atom0 + a, lane); break;
                    default: td_expand_stage<8>(st, al, atom0 + a, lane); break;
                }
            }
        } else {
            // cached-channel stage: fp16 tiles [pool column][256 rows] -> A fragments -> tensor memory
            const int mi = lane >> 3, r = lane & 7;
            const int nsub = min(4, (P_pad - 64 * (it - w.n_w)) >> 4);
            for (int j = 0; j < nsub; ++j) {
#pragma unroll
                for (int a = 0; a < 2; ++a) {
                    uint32_t af[4];
                    const uint32_t addr = smem_u32(st + (j * 16 + (mi >> 1) * 8 + r) * TD_SIG_TILE_STRIDE +
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
    return true;
}

// Fold warps (8..15): same (lane quarter, M tile) mapping, two atoms each.  For every accumulator group
// of every stage: wait for the MMA, read the group back, total += (s * 2^(24-bias)) * acc + m * sum_k x_k
// (cached-channel groups: total += acc), hand the accumulator buffer and then the stage back.
// Register 4j + 2*rowhalf + c of a 16x256b load is (row gid + 8*rowhalf, token 8j + 2*tid4 + c).
template <bool GATEUP, int NJ>
__device__ __forceinline__ bool td_fold_item(const TdParams& p, const TdItem& w, TdBars* B, uint8_t* stages,
                                             float* part, uint32_t tbase, uint32_t& gi, uint32_t& gq, uint32_t ic,
                                             volatile int* poison) {
    const LayerDev* L = p.L;
    int32_t* status = p.ws.status;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q = warp & 3, mt = (warp - TD_W_FOLD) >> 2;
    const int atom0 = 8 * mt + 2 * q;
    const int gid = lane >> 2, tid4 = lane & 3;
    const uint32_t d_lanes = tbase + ((uint32_t)(32 * q) << 16) + 32 * mt;
    const int G = L->G;
    const int bits = w.bits;
    const int code_bytes = block_code_bytes(bits);
    const int xoff = td_xoff_weight(w.blk_bytes);
    const float unscale = __uint_as_float((uint32_t)(127 + 24 - x_scale_bias(bits)) << 23);
    float acc[2][4 * NJ];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int i = 0; i < 4 * NJ; ++i) acc[a][i] = 0.f;
    const int n_it = w.n_w + w.n_ps;
    for (int it = 0; it < n_it; ++it, ++gi) {
        const int s = gi % TD_NS, ph = (gi / TD_NS) & 1;
        if (!mbar_wait_bounded(&B->full[s], ph, poison, status)) return false;  // makes the slot's offset visible
        const uint8_t* st = stages + B->off[s];
        const bool wst = it < w.n_w;
        const int ngrp = wst ? KC / G : 1;
        for (int g = 0; g < ngrp; ++g, ++gq) {
            const int dbuf = gq & 1;
            if (!mbar_wait_bounded(&B->d_full[dbuf], (gq >> 1) & 1, poison, status)) return false;
            tc_fence_after();
            uint32_t r[2][4 * NJ];
#pragma unroll
            for (int a = 0; a < 2; ++a) {
                if constexpr (NJ == 4) tc_ld_x4(d_lanes + ((uint32_t)(16 * a) << 16) + 64 * dbuf, r[a]);
                else tc_ld_x2(d_lanes + ((uint32_t)(16 * a) << 16) + 64 * dbuf, r[a]);
            }
            if (wst) {
                const uint32_t* prm = reinterpret_cast<const uint32_t*>(st + code_bytes);
                float2 xs[NJ];
#pragma unroll
                for (int j = 0; j < NJ; ++j) {
                    const uint8_t* sums = st + xoff + j * TC_RG_STRIDE + TD_SUM_OFF + 2 * tid4 * 4;
                    if (G == 64) {
                        xs[j] = *reinterpret_cast<const float2*>(sums + g * 32);
                    } else {
                        const float2 u = *reinterpret_cast<const float2*>(sums), v = *reinterpret_cast<const float2*>(sums + 32);
                        xs[j] = make_float2(u.x + v.x, u.y + v.y);
                    }
                }
                float s0[2], s1[2], m0[2], m1[2];
#pragma unroll
                for (int a = 0; a < 2; ++a) {
                    const int r0 = 16 * (atom0 + a) + gid;
                    const uint32_t p0 = prm[r0 * ngrp + g], p1 = prm[(r0 + 8) * ngrp + g];
                    const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&p0));
                    const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&p1));
                    s0[a] = f0.x * unscale; s1[a] = f1.x * unscale; m0[a] = f0.y; m1[a] = f1.y;
                }
                tc_wait_ld();
#pragma unroll
                for (int a = 0; a < 2; ++a)
#pragma unroll
                    for (int j = 0; j < NJ; ++j) {
                        acc[a][4 * j + 0] = fmaf(s0[a], __uint_as_float(r[a][4 * j + 0]), fmaf(m0[a], xs[j].x, acc[a][4 * j + 0]));
                        acc[a][4 * j + 1] = fmaf(s0[a], __uint_as_float(r[a][4 * j + 1]), fmaf(m0[a], xs[j].y, acc[a][4 * j + 1]));
                        acc[a][4 * j + 2] = fmaf(s1[a], __uint_as_float(r[a][4 * j + 2]), fmaf(m1[a], xs[j].x, acc[a][4 * j + 2]));
                        acc[a][4 * j + 3] = fmaf(s1[a], __uint_as_float(r[a][4 * j + 3]), fmaf(m1[a], xs[j].y, acc[a][4 * j + 3]));
                    }
            } else {
                tc_wait_ld();
#pragma unroll
                for (int a = 0; a < 2; ++a)
#pragma unroll
                    for (int i = 0; i < 4 * NJ; ++i) acc[a][i] += __uint_as_float(r[a][i]);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&B->d_empty[dbuf]);
        }
        if (lane == 0) mbar_arrive(&B->empty[s]);
    }

    if constexpr (GATEUP) {
        // SwiGLU: register pair (4j + c, 4j + 2 + c) = (gate, up) of hidden index 8*atom + gid, token 8j + 2*tid4 + c.
        // h is rounded to fp16, stored times the power of two the down matrix's codes expect; the sums of
        // the unscaled fp16 values per 64 hidden indices go beside the tile.
#pragma unroll
        for (int a = 0; a < 2; ++a) {
            const int atom = atom0 + a;
            const float scl = __uint_as_float((uint32_t)(127 + x_scale_exp(bits, 8 * atom + gid)) << 23);
            float* mypart = part + ((ic & 1) * 16 + atom) * TD_N;
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int n = 8 * j + 2 * tid4 + c;
                    const float v0 = acc[a][4 * j + c], v1 = acc[a][4 * j + 2 + c];
                    float h16 = 0.f;
                    if (n < w.n_valid) {
                        const float h = v0 / (1.f + expf(-v0)) * v1;
                        h16 = __half2float(__float2half_rn(h));
                        uint8_t* dst = p.ws.hbuf + act_off(w.rb, 8 * (w.rg0 + j), p.ws.Rcap) + atom * 128 +
                                       (2 * tid4 + c) * 16 + gid * 2;
                        *reinterpret_cast<__half*>(dst) = __float2half_rn(h16 * scl);
                    }
                    // sum over the atom's eight hidden indices (lanes of equal tid4), fixed butterfly order
                    float sum = h16;
                    sum += __shfl_xor_sync(0xffffffffu, sum, 4);
                    sum += __shfl_xor_sync(0xffffffffu, sum, 8);
                    sum += __shfl_xor_sync(0xffffffffu, sum, 16);
                    if (gid == 0) mypart[n] = sum;
                }
            }
        }
        // all 16 atoms of the block: add the eight partials of each half chunk in atom order
        // (an mbarrier with a bounded wait, not bar.sync: after an expired wait elsewhere nobody may block here)
        __syncwarp();
        if (lane == 0) mbar_arrive(&B->epi);
        if (!mbar_wait_bounded(&B->epi, ic & 1, poison, status)) return false;
        const int tix = threadIdx.x - TD_W_FOLD * 32;
        if (tix < 2 * 8 * NJ) {
            const int half = tix / (8 * NJ), n = tix % (8 * NJ);
            if (n < w.n_valid) {
                const float* pp = part + ((ic & 1) * 16 + 8 * half) * TD_N + n;
                float sum = 0.f;
#pragma unroll
                for (int a = 0; a < 8; ++a) sum += pp[a * TD_N];
                uint8_t* dst = p.ws.hbuf + act_off(w.rb, 8 * (w.rg0 + (n >> 3)), p.ws.Rcap) + TD_SUM_OFF;
                *reinterpret_cast<float*>(dst + (half * 8 + (n & 7)) * 4) = sum;
            }
        }
    } else {
        float* yb = p.ws.ypart + (size_t)w.split * p.split_stride;
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int n = 8 * j + 2 * tid4 + c;
                    if (n < w.n_valid) {
                        float* yrow = yb + (size_t)(w.row0 + n) * L->d + w.rb * RB + (atom0 + a) * 16 + gid;
                        yrow[0] = acc[a][4 * j + c];
                        yrow[8] = acc[a][4 * j + 2 + c];
                    }
                }
            }
    }
    return true;
}

template <bool GATEUP>
__global__ void __launch_bounds__(TD_THREADS, 1) ffn_tcd_kernel(const TdParams p) {
    extern __shared__ __align__(1024) uint8_t smem[];
    pdl_prologue();
    const LayerDev* L = p.L;
    const int G = L->G;
    const int K = GATEUP ? L->d : L->f;
    const int n_kc = K / KC;
    const int P_pad = L->P_pad;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    TdBars* B = reinterpret_cast<TdBars*>(smem);
    int* prefix = reinterpret_cast<int*>(smem + TD_OFF_PREFIX);
    float* part = reinterpret_cast<float*>(smem + TD_OFF_PART);
    uint8_t* stages = smem + TD_OFF_STAGE;

    // Item table: every expert with rows contributes (token chunks x row blocks x K splits) items.
    for (int i = threadIdx.x; i < p.n_experts; i += TD_THREADS) {
        const int cnt = p.ws.counts[L->order[i]];
        prefix[i + 1] = ((cnt + TD_N - 1) / TD_N) * p.n_rb * p.ksplit;
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
    // Nothing to do, or an earlier wait expired: leave before any tensor memory is allocated.
    if ((int)blockIdx.x >= total || *p.ws.status != STATUS_OK) return;

    if (threadIdx.x == 0) {
        for (int i = 0; i < TD_NS; ++i) {
            mbar_init(&B->full[i], 1);
            mbar_init(&B->empty[i], TD_FOLD_WARPS);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&B->a_full[i], TD_EXP_WARPS);
            mbar_init(&B->a_empty[i], 2);  // both MMA warps commit
            mbar_init(&B->d_full[i], 2);
            mbar_init(&B->d_empty[i], TD_FOLD_WARPS);
        }
        mbar_init(&B->epi, TD_FOLD_WARPS);
        B->poison = 0;
        fence_barrier_init();
    }
    if (warp == TD_W_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&B->tmem_base)),
                     "r"(TD_TMEM_COLS)
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
    // Every role walks the same items (static round-robin over the persistent grid) with its own running
    // stage counter gi (ring slot, A buffer and their phases) and group counter gq (accumulator buffer).
    int cursor = 0;
    uint32_t gi = 0, gq = 0;

    if (warp == TD_W_PROD) {
        // ---------------- producer ----------------
        bool ok = true;
        // byte ring: head = next write offset, tail = oldest stage not yet released, free_b = free bytes
        int head = 0, free_b = TD_RING_BYTES;
        uint32_t tail = 0;
        auto acquire = [&](int need) -> int {  // lane 0 only; returns the ring offset or -1 after an expired wait
            need = (need + 127) & ~127;
            int pad = 0;
            if (head + need > TD_RING_BYTES) {
                pad = TD_RING_BYTES - head;
                head = 0;
            }
            const int tot = need + pad;
            while (free_b < tot || tail + TD_NS <= gi) {
                const int q = tail % TD_NS;
                if (!mbar_wait_bounded(&B->empty[q], (tail / TD_NS) & 1, poison, status)) return -1;
                free_b += B->size[q];
                ++tail;
            }
            const int q = gi % TD_NS;
            B->off[q] = head;
            B->size[q] = tot;
            free_b -= tot;
            const int off = head;
            head += need;
            return off;
        };
        for (int g = blockIdx.x; g < total && ok; g += gridDim.x) {
            const TdItem w = td_decode_item<GATEUP>(p, prefix, g, cursor, n_kc);
            const int n_it = w.n_w + w.n_ps;
            for (int it = 0; it < n_it && ok; ++it, ++gi) {
                const int s = gi % TD_NS;
                // the MMA reads whole 16-token operand tiles: reserve up to that boundary (only n_rg groups are copied)
                const int c0 = 64 * (it - w.n_w), ngr = min(2, (P_pad - c0) >> 5);
                const int xoff = it < w.n_w ? td_xoff_weight(w.blk_bytes) : td_xoff_pool(ngr);
                const int need = it < w.n_w ? xoff + (w.n_mma >> 3) * TC_RG_STRIDE : xoff + ngr * (TD_N / 8) * 512;
                int off = 0;
                if (lane == 0) off = acquire(need);
                off = __shfl_sync(0xffffffffu, off, 0);
                ok = off >= 0;
                if (!ok) break;
                uint8_t* st = stages + off;
                if (lane == 0) {
                    B->xdesc[s] = ((smem_u32(st + xoff) >> 4) & 0x3fffu) | ((128u >> 4) << 16);
                    if (it < w.n_w) {
                        // two copies per stage: the packed block and the operand tile (chunk-major: contiguous)
                        const int kc = w.kc0 + it;
                        mbar_arrive_expect_tx(&B->full[s], (uint32_t)(w.blk_bytes + w.n_rg * TC_RG_STRIDE));
                        bulk_g2s(st, w.wbase + (size_t)kc * w.blk_bytes, (uint32_t)w.blk_bytes, &B->full[s]);
                        bulk_g2s(st + xoff, xbase + act_off(kc, 8 * w.rg0, p.ws.Rcap),
                                 (uint32_t)(w.n_rg * TC_RG_STRIDE), &B->full[s]);
                    } else {
                        // cached-channel stage: up to 64 pool columns = one tile copy + one operand copy per 32 columns
                        mbar_arrive_expect_tx(&B->full[s],
                                              (uint32_t)(ngr * POOL_GROUP * POOL_TILE_PITCH + ngr * w.n_rg * 512));
                        bulk_g2s(st, reinterpret_cast<const uint8_t*>(w.ex->pool_hi) + pool_tile_off(w.rb, c0, P_pad),
                                 (uint32_t)(ngr * POOL_GROUP * POOL_TILE_PITCH), &B->full[s]);
                        for (int j = 0; j < ngr; ++j)
                            bulk_g2s(st + xoff + j * (TD_N / 8) * 512,
                                     reinterpret_cast<const uint8_t*>(p.ws.xsig) +
                                         xpool_off((c0 >> 5) + j, 8 * w.rg0, p.ws.Rcap),
                                     (uint32_t)(w.n_rg * 512), &B->full[s]);
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
    } else if (warp < TD_W_EXP) {
        // ---------------- MMA issuers: four warps = (M tile) x (stage parity) ----------------
        // A tcgen05.mma costs its issuing warp ~50 cycles whatever N is, so one warp cannot feed 16 of them per
        // stage at the rate the weights stream in: each warp issues the 8 MMAs of its M tile for every other
        // stage.  Consecutive stages use different A and accumulator buffers, so the four warps never issue
        // into the same accumulator concurrently.  The code is warp-uniform (one elected lane issues) and
        // short: these warps share their schedulers with the expand and fold warps.
        const int mt = (warp - TD_W_MMA) & 1, par = (warp - TD_W_MMA) >> 1;
        bool ok = true;
        const int ngrp = KC / G;
        for (int g = blockIdx.x; g < total && ok; g += gridDim.x) {
            const TdItem w = td_decode_item<GATEUP>(p, prefix, g, cursor, n_kc);
            const uint32_t idesc = (1u << 4) | ((uint32_t)(w.n_mma >> 3) << 17) | (8u << 24);
            const int n_it = w.n_w + w.n_ps;
            for (int it = 0; it < n_it && ok; ++it, ++gi) {
                const bool wst = it < w.n_w;
                const int my_groups = wst ? ngrp : 1;
                if (TD_MMA_WARPS == 4 && (int)(gi & 1) != par) {
                    gq += my_groups;
                    continue;
                }
                const int s = gi % TD_NS;
                const int b = gi & 1, bph = (gi >> 1) & 1;
                // a published A buffer implies the stage's bytes have landed (the expand warps waited for them)
                int okl = 1;
                if (lane == 0)
                    okl = (mbar_wait_bounded(&B->a_full[b], bph, poison, status) &&
                           mbar_wait_bounded(&B->d_empty[gq & 1], ((gq >> 1) & 1) ^ 1, poison, status))
                              ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, okl, 0) != 0;
                if (!ok) break;
                tc_fence_after();
                // operand descriptor of the stage, prepared by the producer: low word = address | LBO
                const uint64_t desc0 = ((uint64_t)(wst ? TD_DESC_HI_W : TD_DESC_HI_P) << 32) | B->xdesc[s];
                const uint32_t a0 = tbase + TD_COL_A + 128 * b + 64 * mt;
                if (wst) {
                    if (ngrp == 1) {
                        const uint32_t d0 = tbase + 64 * (gq & 1) + 32 * mt;
#pragma unroll
                        for (int k8 = 0; k8 < 8; ++k8)
                            tc_mma_ts_elect(d0, a0 + 8 * k8, desc0 + (uint64_t)(16 * k8), idesc, k8 ? 1u : 0u);
                        tc_commit_elect(&B->d_full[gq & 1]);
                        ++gq;
                    } else {
#pragma unroll
                        for (int gg = 0; gg < 2; ++gg, ++gq) {
                            const int dbuf = gq & 1;
                            if (gg) {  // the second group's buffer: last used by the previous stage
                                int ok2 = 1;
                                if (lane == 0)
                                    ok2 = mbar_wait_bounded(&B->d_empty[dbuf], ((gq >> 1) & 1) ^ 1, poison, status) ? 1 : 0;
                                ok = __shfl_sync(0xffffffffu, ok2, 0) != 0;
                                if (!ok) break;
                                tc_fence_after();
                            }
                            const uint32_t d0 = tbase + 64 * dbuf + 32 * mt;
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4)
                                tc_mma_ts_elect(d0, a0 + 8 * (4 * gg + k4), desc0 + (uint64_t)(16 * (4 * gg + k4)), idesc,
                                                k4 ? 1u : 0u);
                            tc_commit_elect(&B->d_full[dbuf]);
                        }
                        if (!ok) break;
                    }
                } else {
                    const int nsub = min(4, (P_pad - 64 * (it - w.n_w)) >> 4);  // 16-column MMA steps in this stage
                    const uint32_t d0 = tbase + 64 * (gq & 1) + 32 * mt;
                    for (int j = 0; j < nsub; ++j)
                        // operand tile of the 32-column group j/2: [row group][k-octet 4][8][8]; step (j & 1) = two octets
                        tc_mma_ts_elect(d0, a0 + 8 * j, desc0 + (uint64_t)((j >> 1) * ((TD_N / 8) * 512 / 16) + (j & 1) * 16),
                                        idesc, j ? 1u : 0u);
                    tc_commit_elect(&B->d_full[gq & 1]);
                    ++gq;
                }
                tc_commit_elect(&B->a_empty[b]);
            }
        }
    } else {
        // ---------------- expand warps / fold warps ----------------
        bool ok = true;
        uint32_t ic = 0;  // items done by this CTA
        for (int g = blockIdx.x; g < total && ok; g += gridDim.x, ++ic) {
            const TdItem w = td_decode_item<GATEUP>(p, prefix, g, cursor, n_kc);
            if (warp < TD_W_FOLD)
                ok = td_expand_item<GATEUP>(p, w, B, stages, tbase, gi, poison);
            else
                ok = w.n_mma > 16 ? td_fold_item<GATEUP, 4>(p, w, B, stages, part, tbase, gi, gq, ic, poison)
                                  : td_fold_item<GATEUP, 2>(p, w, B, stages, part, tbase, gi, gq, ic, poison);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == TD_W_MMA) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(TD_TMEM_COLS) : "memory");
    }
}

template <bool GATEUP>
static cudaError_t launch_td_one(const TdParams& p, dim3 grid, cudaStream_t st) {
    cudaError_t err =
        cudaFuncSetAttribute(ffn_tcd_kernel<GATEUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, TD_SMEM_BYTES);
    if (err != cudaSuccess) return err;
    return launch_pdl(ffn_tcd_kernel<GATEUP>, grid, dim3(TD_THREADS), (size_t)TD_SMEM_BYTES, st, p);
}

// n_rb: 256-row weight blocks; n_experts: experts in L->order; n_sms: one persistent CTA per SM.
cudaError_t launch_ffn_tcd(const LayerDev* L, const WsDev& ws, int gateup, int n_rb, int ksplit, int n_experts,
                           long long split_stride, int n_sms, cudaStream_t st) {
    TdParams p;
    p.L = L;
    p.ws = ws;
    p.n_rb = n_rb;
    p.n_experts = n_experts;
    p.ksplit = ksplit;
    p.split_stride = split_stride;
    dim3 grid((unsigned)n_sms);
    return gateup ? launch_td_one<true>(p, grid, st) : launch_td_one<false>(p, grid, st);
}

}  // namespace dyn
