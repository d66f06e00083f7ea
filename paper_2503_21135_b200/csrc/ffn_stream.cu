// Streaming grouped dequant-GEMM for small token counts per expert (decode path, and the generic
// fallback for any size): HBM-bound, judged on packed-weight bytes per second.
//
// PERSISTENT grid (two or three CTAs per SM).  A work item = one (expert, 256-row weight block, chunk of <= 24
// tokens, K split); items are ordered costliest first (most 8-token tiles first from 33 rows per expert on, then
// heaviest bit-width) and handed out from a device counter, a CTA's first item statically.  Inside a CTA ONE
// producer thread streams the packed blocks (codes + params, contiguous per 256 x 128 block) and the matching
// activation slices into a shared-memory ring with bulk async copies completing on mbarriers; it runs ahead across
// item boundaries, so the ring never drains between items.  The group size is a template parameter (the group
// bookkeeping of the inner loop folds away).  Eight consumer warps, each owning two 16-row atoms, turn codes into fp16
// operands with ONE logic op per register pair: a code field masked in place at bit offset o is the
// fp16 subnormal q * 2^(o-24), and the activation slice already carries the factor 2^(bias-o) (see
// layout.cuh).  They issue mma.sync m16n8k16 (weights = A, tokens = B, fp32 accumulate) and apply
// scale / zero once per group after the dot product:
//     sum_k (s*q_k + m) x_k = (s * 2^(24-bias)) * acc + m * sum_k x_k .
// The per-group sums of x come precomputed with the activation slice.  Codes and activations are
// exact in fp16, so the only roundings are the fp32 accumulation and the fp16 rounding of h.
// The number of 8-token tiles (1..3) is chosen per item from the expert's actual token count.
//
// Gate/up items: after the K loop the significant-channel correction runs as extra ring stages
// (16 channels each): the fp16 tiles of the active cached channels are fetched through the slot ->
// pool-position table and multiplied with the gathered activation columns into the same
// accumulators; then SwiGLU, fp16 rounding of h, per-64 sums of h, coalesced store of h (scaled
// for the down matrix).  Down items: fp32 partial outputs per K split.
#include <type_traits>

#include "common.cuh"
#include "expand.cuh"
#include "layout.cuh"

namespace dyn {

constexpr int APW = 2;                 // atoms (16 weight rows) per consumer warp (1 = sixteen consumer warps at 56
                                       // registers: 197 vs 171 us on the gate/up launch at 64 tokens, 124 vs 103 at 8)
constexpr int CONSUMER_WARPS = 16 / APW;
constexpr int FFN_THREADS = (CONSUMER_WARPS + 1) * 32;
constexpr int SMEM_HEADER = 2048;     // barriers, poison flag, per-expert item prefix table
constexpr int MAX_STAGES = 16;        // ring queue depth; the ring itself is byte-granular
// Tokens per work item.  24, not 32: with at most three 8-token tiles the two accumulator sets of a warp fit the 96
// registers that two resident CTAs leave a thread (four tiles spilled ~1.3 KB of loads per thread into the
// loops); an expert of 25-32 rows takes a second, short pass over its blocks, which hits L2.
constexpr int CHUNK_TOKENS = 24;

struct FfnParams {
    const LayerDev* L;
    WsDev ws;
    int ksplit;
    long long split_stride;  // elements between K-split partial outputs
    int smem_bytes;
    int ring_bytes;          // bytes of the stage ring (stages take what they need, in order)
    int htile_bytes;         // bytes of one h tile behind the ring
    int n_rb;                // 256-row weight blocks of the matrix
    int n_experts;
    int32_t* work_ctr;       // device counter of this launch's work queue (zeroed by the scan kernel)
    int sectioned;           // items ordered by tile count first (batches where an expert can have more than 32 rows)
};

struct Item {
    int e, rb, split, row0, nvalid;
};

struct FfnSmem {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], done;
    int off[MAX_STAGES];    // ring offset of the stage in queue slot q (written by the producer before it arrives)
    int size[MAX_STAGES];   // bytes the stage holds in the ring (producer only)
    int first_item[MAX_STAGES];  // item index if the stage opens an item, -2 if not, -1: no more items
    volatile int poison;
    int n_items;
    // Item order.  Sectioned (up to MAX_SECT_EXPERTS experts): three sections by the number of 8-token tiles of an
    // item's token chunk (3, 2, 1: the time of a pipeline stage grows with it, and the costliest items go first so
    // that the CTAs finish together), inside a section experts by descending bit-width; prefix[sec * (n + 1) + y] =
    // items of the section before expert order[y], sec_base[sec] = first item of the section.  Otherwise one section
    // with every chunk of an expert (prefix[y]).
    int sectioned;
    int sec_base[4];
    int prefix[MAX_EXPERTS + 1];
};
constexpr int MAX_SECT_EXPERTS = (MAX_EXPERTS + 1) / 3 - 1;
static_assert(sizeof(FfnSmem) <= SMEM_HEADER, "header too small");

// Decode item index g into (expert, row block, split, token chunk).  The cursor only moves forward (item indices
// come in ascending order).
struct Cursor {
    int sec = 0, y = 0;
};
template <bool SECT>
__device__ __forceinline__ Item decode_item(const FfnParams& p, const FfnSmem* S, int g, Cursor& cur) {
    int e, cnt, tc, rbs;
    if (SECT && S->sectioned) {
        const int sec = g < S->sec_base[1] ? 0 : (g < S->sec_base[2] ? 1 : 2);
        if (sec != cur.sec) {
            cur.sec = sec;
            cur.y = 0;
        }
        const int* pr = S->prefix + sec * (p.n_experts + 1);
        const int gl = g - S->sec_base[sec];
        while (gl >= pr[cur.y + 1]) ++cur.y;
        e = p.L->order[cur.y];
        cnt = p.ws.counts[e];
        const int n_full = cnt / CHUNK_TOKENS, rem_tiles = (cnt % CHUNK_TOKENS + 7) >> 3;
        const int local = gl - pr[cur.y];
        if (sec == 0) {  // the chunks of three tiles: the full ones and a remainder of 17..23 tokens
            const int n3 = n_full + (rem_tiles == 3 ? 1 : 0);
            tc = local % n3;   // chunks of one weight block are neighbours: they share L2 lines
            rbs = local / n3;
        } else {         // the remainder chunk
            tc = n_full;
            rbs = local;
        }
    } else {
        while (g >= S->prefix[cur.y + 1]) ++cur.y;
        e = p.L->order[cur.y];
        cnt = p.ws.counts[e];
        const int n_tc = (cnt + CHUNK_TOKENS - 1) / CHUNK_TOKENS;
        const int local = g - S->prefix[cur.y];
        tc = local % n_tc;
        rbs = local / n_tc;
    }
    Item it;
    it.e = e;
    it.rb = rbs / p.ksplit;
    it.split = rbs % p.ksplit;
    it.row0 = p.ws.off_pad[e] + tc * CHUNK_TOKENS;
    it.nvalid = min(CHUNK_TOKENS, cnt - tc * CHUNK_TOKENS);
    return it;
}

// m16n8k16 with a zero C operand: d = a * b
__device__ __forceinline__ void mma16816_z(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}

// Consumer side of one work item.  `stage_it` is the CTA-wide ring position, `item_idx` the number of
// items this CTA has finished (parity of the epilogue barrier / h tile).
template <int BITS, int NT8, bool GATEUP, int G>
__device__ __forceinline__ bool consume_item(const FfnParams& p, FfnSmem* S, uint8_t* stages, uint8_t* htiles,
                                             const Item& im, int& stage_it, int item_idx, bool& clamped) {
    constexpr int NS = MAX_STAGES;
    const LayerDev* L = p.L;
    const ExpertDev& ex = L->ex[im.e];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tid4 = lane & 3;
    const int atom0 = warp * APW;
    const int K = GATEUP ? L->d : L->f;
    const int n_kc = K / KC;
    constexpr int code_bytes = 4096 * BITS;
    constexpr int blk_bytes = code_bytes + RB * (KC / G) * 4;   // = block_bytes(BITS, G), the expert's blk_bytes
    int kc0 = 0, kc1 = n_kc;
    if (!GATEUP) {
        kc0 = (int)(((long long)im.split * n_kc) / p.ksplit);
        kc1 = (int)(((long long)(im.split + 1) * n_kc) / p.ksplit);
    }
    const int sig_cnt = (GATEUP && ex.switchable) ? L->sig_cnt[im.e] : 0;
    const int n_ps = sig_cnt > 0 ? (L->P_pad >> 5) : 0;
    volatile int* poison = &S->poison;

    float total[APW][NT8][4];
#pragma unroll
    for (int a = 0; a < APW; ++a)
#pragma unroll
        for (int j = 0; j < NT8; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) total[a][j][c] = 0.f;

    // exact power of two that undoes the operand scaling: codes enter as q*2^(o-24), activations as x*2^(bias-o)
    const float unscale = __uint_as_float((uint32_t)(127 + 24 - x_scale_bias(BITS)) << 23);
    constexpr int ngrp = KC / G;

    for (int kc = kc0; kc < kc1; ++kc, ++stage_it) {
        const int s = stage_it % NS, ph = (stage_it / NS) & 1;
        if (!mbar_wait_bounded(&S->full[s], ph, poison, p.ws.status)) return false;
        const uint8_t* st = stages + S->off[s];
        const uint8_t* xs = st + blk_bytes;
        const uint32_t* prm = reinterpret_cast<const uint32_t*>(st + code_bytes);
        float accg[APW][NT8][4];   // the first MMA of a quantization group starts from a zero C operand

#pragma unroll
        for (int half = 0; half < 2; ++half) {
            Codes<BITS> cd[APW];
#pragma unroll
            for (int a = 0; a < APW; ++a) load_codes<BITS>(cd[a], st + (atom0 + a) * atom_bytes(BITS), lane, half);

            auto step = [&](auto S4c, auto firstc) {
                constexpr int S4 = decltype(S4c)::value;
                constexpr bool FIRST = decltype(firstc)::value;
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
                for (int a = 0; a < APW; ++a) {
                    uint32_t af[4];
                    expand<BITS, S4>(cd[a], af);
#pragma unroll
                    for (int j = 0; j < NT8; ++j) {
                        if constexpr (FIRST) mma16816_z(accg[a][j], af, b0[j], b1[j]);
                        else mma16816(accg[a][j], af, b0[j], b1[j]);
                    }
                }
            };
            if (G == 64 || half == 0) step(std::integral_constant<int, 0>{}, std::true_type{});
            else step(std::integral_constant<int, 0>{}, std::false_type{});
            step(std::integral_constant<int, 1>{}, std::false_type{});
            step(std::integral_constant<int, 2>{}, std::false_type{});
            step(std::integral_constant<int, 3>{}, std::false_type{});

            if (G == 64 || half == 1) {
                // fold the group: total += (s * unscale) * acc + m * sum(x); two FMAs per element
                const int g = (G == 64) ? half : 0;
                float xs0[NT8], xs1[NT8];
#pragma unroll
                for (int j = 0; j < NT8; ++j) {
                    const float2 sa = *reinterpret_cast<const float2*>(xs + (8 * j + 2 * tid4) * XROW + XROW_SUM_OFF);
                    const float2 sb = *reinterpret_cast<const float2*>(xs + (8 * j + 2 * tid4 + 1) * XROW + XROW_SUM_OFF);
                    if (G == 64) { xs0[j] = half ? sa.y : sa.x; xs1[j] = half ? sb.y : sb.x; }
                    else { xs0[j] = sa.x + sa.y; xs1[j] = sb.x + sb.y; }
                }
#pragma unroll
                for (int a = 0; a < APW; ++a) {
                    const int r0 = (atom0 + a) * 16 + gid;
                    const uint32_t p0 = prm[r0 * ngrp + g], p1 = prm[(r0 + 8) * ngrp + g];
                    const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&p0));
                    const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&p1));
                    const float s0 = f0.x * unscale, s1 = f1.x * unscale;
#pragma unroll
                    for (int j = 0; j < NT8; ++j) {
                        total[a][j][0] = fmaf(s0, accg[a][j][0], fmaf(f0.y, xs0[j], total[a][j][0]));
                        total[a][j][1] = fmaf(s0, accg[a][j][1], fmaf(f0.y, xs1[j], total[a][j][1]));
                        total[a][j][2] = fmaf(s1, accg[a][j][2], fmaf(f1.y, xs0[j], total[a][j][2]));
                        total[a][j][3] = fmaf(s1, accg[a][j][3], fmaf(f1.y, xs1[j], total[a][j][3]));
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&S->empty[s]);
    }

    if constexpr (GATEUP) {
        // cached-channel stages: the 8-bit-valued tiles of 32 pool columns times their activations (zero for
        // channels that are not significant right now), accumulated straight into the totals
        for (int ps = 0; ps < n_ps; ++ps, ++stage_it) {
            const int s = stage_it % NS, ph = (stage_it / NS) & 1;
            if (!mbar_wait_bounded(&S->full[s], ph, poison, p.ws.status)) return false;
            const uint8_t* st = stages + S->off[s];
            const uint8_t* xs = st + POOL_GROUP * POOL_TILE_PITCH;
            const int mi = lane >> 3, r = lane & 7;
#pragma unroll
            for (int ks = 0; ks < POOL_GROUP / 16; ++ks) {
                uint32_t b0[NT8], b1[NT8];
#pragma unroll
                for (int j = 0; j < NT8; ++j) {
                    b0[j] = *reinterpret_cast<const uint32_t*>(xs + (8 * j + gid) * XPOOL_ROW + (16 * ks + 2 * tid4) * 2);
                    b1[j] = *reinterpret_cast<const uint32_t*>(xs + (8 * j + gid) * XPOOL_ROW + (16 * ks + 2 * tid4 + 8) * 2);
                }
#pragma unroll
                for (int a = 0; a < APW; ++a) {
                    uint32_t af[4];
                    const uint32_t addr = smem_u32(st + (16 * ks + (mi >> 1) * 8 + r) * POOL_TILE_PITCH +
                                                   (16 * (atom0 + a) + (mi & 1) * 8) * 2);
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(af[0]), "=r"(af[1]), "=r"(af[2]), "=r"(af[3])
                                 : "r"(addr));
#pragma unroll
                    for (int j = 0; j < NT8; ++j) mma16816(total[a][j], af, b0[j], b1[j]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&S->empty[s]);
        }
    }

    if constexpr (GATEUP) {
        // SwiGLU: rows 0..7 of an atom are gate, rows 8..15 the matching up rows.
        uint8_t* htile = htiles + (item_idx & 1) * p.htile_bytes;
#pragma unroll
        for (int a = 0; a < APW; ++a)
#pragma unroll
            for (int j = 0; j < NT8; ++j)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const float g = total[a][j][c], u = total[a][j][2 + c];
                    float h = g / (1.f + expf(-g)) * u;
                    const int tok = 8 * j + 2 * tid4 + c;
                    if (tok < im.nvalid) h = clamp_act(h, clamped);   // columns past the last token hold stale data
                    h = round_operand(h, p.ws.h_bf16);
                    *reinterpret_cast<__half*>(htile + tok * XROW + (8 * (atom0 + a) + gid) * 2) = __float2half_rn(h);
                }
        __syncwarp();
        if (lane == 0) mbar_arrive(&S->done);
        if (!mbar_wait_bounded(&S->done, item_idx & 1, poison, p.ws.status)) return false;
        // this lane's four hidden indices 4*lane + {0..3}: the down matrix wants them scaled by 2^(bias-o)
        const float sc0 = __uint_as_float((uint32_t)(127 + x_scale_exp(BITS, 4 * lane)) << 23);
        const float sc1 = __uint_as_float((uint32_t)(127 + x_scale_exp(BITS, 4 * lane + 2)) << 23);
        for (int tok = warp; tok < im.nvalid; tok += CONSUMER_WARPS) {
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
            uint8_t* dst = p.ws.hbuf + act_off(im.rb, im.row0 + tok, p.ws.Rcap);
            *reinterpret_cast<uint2*>(dst + lane * 8) = ov;
            if ((lane & 15) == 0) *reinterpret_cast<float*>(dst + XROW_SUM_OFF + (lane >> 4) * 4) = sum;
        }
    } else {
        float* yb = p.ws.ypart + (size_t)im.split * p.split_stride;
        const int d = L->d;
#pragma unroll
        for (int a = 0; a < APW; ++a)
#pragma unroll
            for (int j = 0; j < NT8; ++j)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int tok = 8 * j + 2 * tid4 + (c & 1);
                    const int n = im.rb * RB + (atom0 + a) * 16 + gid + ((c >> 1) ? 8 : 0);
                    if (tok < im.nvalid) yb[(size_t)(im.row0 + tok) * d + n] = total[a][j][c];
                }
    }
    return true;
}

// MAXNT8: most 8-token tiles an item can have in this launch (the host knows the token count): the small
// variants need fewer registers and run three CTAs per SM.
template <int BITS, bool GATEUP, int MAXNT8, int G>
__device__ __forceinline__ bool consume_dispatch(const FfnParams& p, FfnSmem* S, uint8_t* stages, uint8_t* htiles,
                                                 const Item& im, int& stage_it, int item_idx, bool& clamped) {
    const int nt8 = (im.nvalid + 7) >> 3;
    if (MAXNT8 == 1 || nt8 == 1) return consume_item<BITS, 1, GATEUP, G>(p, S, stages, htiles, im, stage_it, item_idx, clamped);
    if constexpr (MAXNT8 >= 2) {
        if (MAXNT8 == 2 || nt8 == 2)
            return consume_item<BITS, 2, GATEUP, G>(p, S, stages, htiles, im, stage_it, item_idx, clamped);
    }
    if constexpr (MAXNT8 >= 3) return consume_item<BITS, 3, GATEUP, G>(p, S, stages, htiles, im, stage_it, item_idx, clamped);
    return false;
}

template <bool GATEUP, int MAXNT8, int G>
__global__ void __launch_bounds__(FFN_THREADS, (MAXNT8 <= 2 && APW == 2) ? 3 : 2) ffn_stream_kernel(const FfnParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    pdl_prologue();
    if (*p.ws.status & STATUS_TIMEOUT) return;  // after an expired wait nothing new starts
    const LayerDev* L = p.L;
    FfnSmem* S = reinterpret_cast<FfnSmem*>(smem);
    uint8_t* stages = smem + SMEM_HEADER;
    constexpr int NS = MAX_STAGES;
    uint8_t* htiles = stages + p.ring_bytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(&S->full[s], 1);
            mbar_init(&S->empty[s], CONSUMER_WARPS);
        }
        mbar_init(&S->done, CONSUMER_WARPS);
        S->poison = 0;
        // items per expert, heaviest bit-width first; experts above tc_min rows take the tcgen05 path
        const int per_chunk = p.n_rb * p.ksplit;
        if (MAXNT8 == 3 && p.sectioned) {
            const int n1 = p.n_experts + 1;
            int acc[3] = {0, 0, 0};   // sections: chunks of 3, 2, 1 tiles
            for (int y = 0; y < p.n_experts; ++y) {
                S->prefix[y] = acc[0];
                S->prefix[n1 + y] = acc[1];
                S->prefix[2 * n1 + y] = acc[2];
                const int cnt = p.ws.counts[L->order[y]];
                if (cnt > 0 && cnt <= p.ws.tc_min) {
                    const int rem_tiles = (cnt % CHUNK_TOKENS + 7) >> 3;
                    acc[0] += (cnt / CHUNK_TOKENS + (rem_tiles == 3 ? 1 : 0)) * per_chunk;
                    if (rem_tiles == 2) acc[1] += per_chunk;
                    if (rem_tiles == 1) acc[2] += per_chunk;
                }
            }
            S->prefix[p.n_experts] = acc[0];
            S->prefix[n1 + p.n_experts] = acc[1];
            S->prefix[2 * n1 + p.n_experts] = acc[2];
            S->sec_base[0] = 0;
            S->sec_base[1] = acc[0];
            S->sec_base[2] = acc[0] + acc[1];
            S->sec_base[3] = acc[0] + acc[1] + acc[2];
            S->n_items = acc[0] + acc[1] + acc[2];
            S->sectioned = 1;
        } else {
            int acc = 0;
            for (int y = 0; y < p.n_experts; ++y) {
                S->prefix[y] = acc;
                const int cnt = p.ws.counts[L->order[y]];
                if (cnt > 0 && cnt <= p.ws.tc_min) acc += ((cnt + CHUNK_TOKENS - 1) / CHUNK_TOKENS) * per_chunk;
            }
            S->prefix[p.n_experts] = acc;
            S->n_items = acc;
            S->sectioned = 0;
        }
        fence_barrier_init();
    }
    __syncthreads();
    const int n_items = S->n_items;
    volatile int* poison = &S->poison;

    if (warp == CONSUMER_WARPS) {
        // ---------------- producer: ONE thread, running ahead across items.  The schedulers share the issue slots among
        // all ready warps, so every instruction of the producer's per-stage path waits its turn behind the consumer
        // warps of three CTAs (a per-stage timeline showed half a microsecond per stage, as long as the consumers need
        // for it): the path is kept as short as it gets, with no warp-wide shuffles or barriers in it ----------------
        if (lane != 0) return;
        int it = 0;
        Cursor y;
        bool ok = true;
        // byte ring: head = next write offset, tail = oldest stage not yet released, free_b = free bytes
        int head = 0, tail = 0, free_b = p.ring_bytes;
        auto acquire = [&](int need) -> int {   // returns the ring offset or -1 after an expired wait
            need = (need + 127) & ~127;
            int pad = 0;
            if (head + need > p.ring_bytes) { pad = p.ring_bytes - head; head = 0; }
            // a stage that wraps while the write offset is still inside its own footprint needs the whole ring
            // (its footprint and the skipped tail overlap): then it waits for every earlier stage and takes it all
            const int total = need + pad < p.ring_bytes ? need + pad : p.ring_bytes;
            while (free_b < total || tail + NS <= it) {
                const int q = tail % NS;
                if (!mbar_wait_bounded(&S->empty[q], (tail / NS) & 1, poison, p.ws.status)) return -1;
                free_b += S->size[q];
                ++tail;
            }
            const int q = it % NS;
            S->off[q] = head;
            S->size[q] = total;
            free_b -= total;
            const int off = head;
            head += need;
            return off;
        };
        const int K = GATEUP ? L->d : L->f;
        const int n_kc = K / KC;
        // Work queue: items are numbered heaviest bit-width first and handed out one at a time (an atomic counter),
        // so a CTA that drew a light item comes back sooner: with one to three items per CTA and items that differ
        // fourfold in bytes, a static deal leaves the CTAs with the 8-bit items far behind the rest.
        bool first_draw = true;
        const bool all_static = n_items <= (int)gridDim.x;  // at most one item per CTA
        while (ok) {
            // the first item of every CTA is dealt statically (CTA j takes item j: one per SM before any SM gets a
            // second one, which matters when there are fewer items than CTAs), the rest come from the counter
            int g = blockIdx.x;
            if (!first_draw) {
                if (all_static) break;  // every item was dealt statically: the consumers know, nothing to signal
                g = gridDim.x + atomicAdd(p.work_ctr, 1);
            } else if (all_static && g >= n_items) {
                break;
            }
            first_draw = false;
            if (g >= n_items) {  // tell the consumers: an empty stage marked -1
                const int off = acquire(128);
                if (off >= 0) {
                    S->first_item[it % NS] = -1;
                    mbar_arrive(&S->full[it % NS]);
                }
                break;
            }
            bool first = true;
            const Item im = decode_item<MAXNT8 == 3>(p, S, g, y);
            const ExpertDev& ex = L->ex[im.e];
            const int blk_bytes = ex.blk_bytes;
            int kc0 = 0, kc1 = n_kc;
            if (!GATEUP) {
                kc0 = (int)(((long long)im.split * n_kc) / p.ksplit);
                kc1 = (int)(((long long)(im.split + 1) * n_kc) / p.ksplit);
            }
            const uint8_t* wbase = (GATEUP ? ex.w13 : ex.w2) + (size_t)im.rb * n_kc * blk_bytes;
            const uint8_t* xbuf = GATEUP ? p.ws.xperm : p.ws.hbuf;
            const int stage_need = blk_bytes + ((im.nvalid + 7) & ~7) * XROW;
            const uint32_t x_bytes = (uint32_t)(im.nvalid * XROW), stage_tx = (uint32_t)blk_bytes + x_bytes;
            const uint8_t* wsrc = wbase + (size_t)kc0 * blk_bytes;
            const uint8_t* xsrc = xbuf + act_off(kc0, im.row0, p.ws.Rcap);
            const size_t x_stride = act_off(1, 0, p.ws.Rcap);   // one k chunk further in the chunk-major buffer
            for (int kc = kc0; kc < kc1 && ok; ++kc, ++it) {
                const int s = it % NS;
                // the consumers read whole 8-token tiles: reserve rows up to the tile boundary (only nvalid are copied)
                const int off = acquire(stage_need);
                ok = off >= 0;
                if (!ok) break;
                uint8_t* st = stages + off;
                // two copies per stage: the packed block and the (chunk-major, hence contiguous) activation slice
                S->first_item[s] = first ? g : -2;
                mbar_arrive_expect_tx(&S->full[s], stage_tx);
                bulk_g2s(st, wsrc, (uint32_t)blk_bytes, &S->full[s]);
                bulk_g2s(st + blk_bytes, xsrc, x_bytes, &S->full[s]);
                wsrc += blk_bytes;
                xsrc += x_stride;
                first = false;
            }
            if constexpr (GATEUP) {
                // cached-channel stages: 32 pool columns each = one 16.9 KB tile copy + one activation copy
                const int n_ps = (ex.switchable && L->sig_cnt[im.e] > 0) ? (L->P_pad >> 5) : 0;
                for (int ps = 0; ps < n_ps && ok; ++ps, ++it) {
                    const int s = it % NS;
                    const int off = acquire(POOL_GROUP * POOL_TILE_PITCH + ((im.nvalid + 7) & ~7) * XPOOL_ROW);
                    ok = off >= 0;
                    if (!ok) break;
                    uint8_t* st = stages + off;
                    S->first_item[s] = -2;
                    mbar_arrive_expect_tx(&S->full[s], (uint32_t)(POOL_GROUP * POOL_TILE_PITCH + im.nvalid * XPOOL_ROW));
                    bulk_g2s(st, reinterpret_cast<const uint8_t*>(ex.pool_hi) + pool_tile_off(im.rb, ps * POOL_GROUP, L->P_pad),
                             POOL_GROUP * POOL_TILE_PITCH, &S->full[s]);
                    bulk_g2s(st + POOL_GROUP * POOL_TILE_PITCH,
                             reinterpret_cast<const uint8_t*>(p.ws.xsig) + xpool_off(ps, im.row0, p.ws.Rcap),
                             (uint32_t)(im.nvalid * XPOOL_ROW), &S->full[s]);
                }
            }
        }
        if (!ok) {
            // gave up: let copies already issued land before the CTA's shared memory is released
            const unsigned long long t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 2000000ull) {
            }
        }
        return;
    }

    // ---------------- consumer warps ----------------
    int stage_it = 0, item_idx = 0;
    Cursor y;
    bool clamped = false;
    const bool all_static = n_items <= (int)gridDim.x;
    for (;; ++item_idx) {
        if (all_static && (item_idx > 0 || (int)blockIdx.x >= n_items)) break;
        // the next stage opens the next item (or says there is none): its index rides with the stage
        int g = blockIdx.x;  // the first item is dealt statically: decode it while its first stage is in flight
        if (item_idx > 0) {
            const int s0 = stage_it % NS;
            if (!mbar_wait_bounded(&S->full[s0], (stage_it / NS) & 1, poison, p.ws.status)) return;
            g = S->first_item[s0];
        }
        if (g < 0 || g >= n_items) break;
        const Item im = decode_item<MAXNT8 == 3>(p, S, g, y);
        bool ok;
        switch (L->ex[im.e].bits) {
            case 2: ok = consume_dispatch<2, GATEUP, MAXNT8, G>(p, S, stages, htiles, im, stage_it, item_idx, clamped); break;
            case 3: ok = consume_dispatch<3, GATEUP, MAXNT8, G>(p, S, stages, htiles, im, stage_it, item_idx, clamped); break;
            case 4: ok = consume_dispatch<4, GATEUP, MAXNT8, G>(p, S, stages, htiles, im, stage_it, item_idx, clamped); break;
            case 6: ok = consume_dispatch<6, GATEUP, MAXNT8, G>(p, S, stages, htiles, im, stage_it, item_idx, clamped); break;
            default: ok = consume_dispatch<8, GATEUP, MAXNT8, G>(p, S, stages, htiles, im, stage_it, item_idx, clamped); break;
        }
        if (!ok) {  // poisoned: the status word says so; keep arriving so that nobody waits on this warp forever
            if (GATEUP && lane == 0) mbar_arrive(&S->done);
            return;
        }
    }
    if (clamped) atomicOr(p.ws.status, STATUS_RANGE);
}

template <bool GATEUP, int MAXNT8, int G>
static cudaError_t launch_one_g(const FfnParams& p, int n_ctas, cudaStream_t st) {
    cudaError_t err = cudaFuncSetAttribute(ffn_stream_kernel<GATEUP, MAXNT8, G>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, p.smem_bytes);
    if (err != cudaSuccess) return err;
    return launch_pdl(ffn_stream_kernel<GATEUP, MAXNT8, G>, dim3((unsigned)n_ctas), dim3(FFN_THREADS),
                      (size_t)p.smem_bytes, st, p);
}
// The group size (64 or 128) is a template parameter: the group bookkeeping of the inner loop folds away.
template <bool GATEUP, int MAXNT8>
static cudaError_t launch_one(const FfnParams& p, int n_ctas, int G, cudaStream_t st) {
    return G == 64 ? launch_one_g<GATEUP, MAXNT8, 64>(p, n_ctas, st) : launch_one_g<GATEUP, MAXNT8, 128>(p, n_ctas, st);
}

// max_rows: upper bound of the rows one expert can have in this forward (selects the kernel variant);
// n_sms: SM count (the persistent grid is 2 or 3 CTAs per SM).
cudaError_t launch_ffn_stream(const LayerDev* L, const WsDev& ws, int gateup, int n_rb, int ksplit, int n_experts,
                              long long split_stride, int max_rows, int n_sms, int G, cudaStream_t st) {
    // three CTAs per SM pay off once every CTA has several items to walk; at 1-3 tokens a CTA sees one or two
    const bool small = max_rows >= 4 && max_rows <= 16;
    const bool three = small && APW == 2;
    const int smem_bytes = three ? 74 * 1024 : 110 * 1024;
    const int n_ctas = (three ? 3 : 2) * n_sms;
    FfnParams p;
    p.L = L;
    p.ws = ws;
    p.ksplit = ksplit;
    p.split_stride = split_stride;
    p.smem_bytes = smem_bytes;
    // two h tiles (double-buffered across items) behind the ring; the small variants hold at most 16 tokens
    p.htile_bytes = (small ? 16 : CHUNK_TOKENS) * XROW;
    p.ring_bytes = (smem_bytes - SMEM_HEADER - (gateup ? 2 * p.htile_bytes : 0)) & ~127;
    p.n_rb = n_rb;
    p.n_experts = n_experts;
    p.work_ctr = ws.status + (gateup ? 4 : 5);
    p.sectioned = (max_rows > 32 && n_experts <= MAX_SECT_EXPERTS) ? 1 : 0;   // measured: +3 % at 64 tokens, -1 % at 32
    if (small && max_rows <= 8) return gateup ? launch_one<true, 1>(p, n_ctas, G, st) : launch_one<false, 1>(p, n_ctas, G, st);
    if (small) return gateup ? launch_one<true, 2>(p, n_ctas, G, st) : launch_one<false, 2>(p, n_ctas, G, st);
    return gateup ? launch_one<true, 3>(p, n_ctas, G, st) : launch_one<false, 3>(p, n_ctas, G, st);
}

}  // namespace dyn
