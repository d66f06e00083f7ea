// Host side of the C-ABI: context, arena / workspace layout, argument validation, launches.
#include <algorithm>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/dynamo.h"
#include "common.cuh"

namespace dyn {
cudaError_t launch_pack_blocks(const void* src_a, const void* src_b, int n_rows_blocks, int K, int G, int bits,
                               int fused, void* dst, cudaStream_t st);
cudaError_t launch_pack_hi(const void* w_gate, const void* w_up, int f, int d, int G, int P,
                           const int32_t* cache_idx_dev, const ExpertDev& ex, cudaStream_t st);
cudaError_t launch_requant(const LayerDev* L, int f, const int32_t* items_dev, int n_items, cudaStream_t st);
cudaError_t launch_retarget(LayerDev* L, int e, int f, int bits, cudaStream_t st);
cudaError_t launch_pack_down_hi(const void* w_down, int d, int f, int G, int P2, const int32_t* cache_idx_dev,
                                int base_bits, const DownExpertDev& ex, cudaStream_t st);
cudaError_t launch_down_fix(const LayerDev* L, const DownDev* D2, const WsDev& ws, int d, cudaStream_t st);
cudaError_t launch_retarget_down(int d, int f, int G, int P2, const int32_t* cache_idx_dev, int base_bits, int hi_bits,
                                 const DownExpertDev& ex, cudaStream_t st);
cudaError_t launch_requant_down(const LayerDev* L, const DownDev* D2, const int32_t* hi_bits_dev, int d, int n_experts,
                                cudaStream_t st);
cudaError_t launch_export_down(const LayerDev* L, const DownDev* D2, int e, int which, long long n_elems, uint8_t* q,
                               uint16_t* sc, uint16_t* zr, cudaStream_t st);
cudaError_t launch_export(const LayerDev* L, int e, int mat, int which, long long n_elems, uint8_t* q, uint16_t* sc,
                          uint16_t* zr, cudaStream_t st);
cudaError_t launch_route(const float* logits, int T, int E, int k, int renorm, int32_t* idx, float* w,
                         cudaStream_t st);
cudaError_t launch_route_gemm(const void* x, const void* w_router, const float* bias, int T, int d, int E, int k,
                              int renorm, float* logits_out, int32_t* idx, float* w, cudaStream_t st);
cudaError_t launch_scan(const WsDev& ws, int E, int Es, int k, cudaStream_t st);
cudaError_t launch_gather(const LayerDev* L, const WsDev& ws, const void* x, cudaStream_t st);
bool front_fits(int T, int k);
cudaError_t launch_front(const LayerDev* L, const WsDev& ws, const void* x, const float* logits, int E, int Es, int k,
                         int renorm, cudaStream_t st);
cudaError_t launch_combine(const WsDev& ws, int d, int k, int Es, void* y, int y_f32, long long split_stride,
                           cudaStream_t st);
cudaError_t launch_ffn_stream(const LayerDev* L, const WsDev& ws, int gateup, int n_rb, int ksplit, int n_experts,
                              long long split_stride, int max_rows, int n_sms, int G, cudaStream_t st);
cudaError_t setup_ffn_tc2(int n_sms, int* clusters_out);
cudaError_t launch_ffn_tc2(const LayerDev* L, const WsDev& ws, int gateup, int n_rb, int n_experts, int n_clusters,
                           cudaStream_t st);
cudaError_t launch_stats(const LayerDev* L, const WsDev& ws, const void* x, float* stats, float* part, int32_t* ctr, int E,
                         int n_slices, cudaStream_t st);
cudaError_t launch_select(const LayerDev* L, float* stats, int E, int P, int n_sel, int reset, int32_t* chosen,
                          cudaStream_t st);
cudaError_t launch_expire_wait(int32_t* status, unsigned long long limit_ns, cudaStream_t st);
cudaError_t launch_switch(const SwitchLayers& layers, int n_layers, int E, const int32_t* staging, int per_layer_ints,
                          cudaStream_t st);
}  // namespace dyn

using namespace dyn;

namespace {

constexpr size_t ALIGN = 256;
constexpr int ROW_PAD = 32;            // extra activation rows so a token chunk may read past the last row
constexpr int MAX_SWITCH_LAYERS = 64;
constexpr int DECODE_ROWS = 1024;      // up to this many permuted rows the down GEMM is split along K
constexpr int MAX_KSPLIT = 8;

inline size_t align_up(size_t v) { return (v + ALIGN - 1) / ALIGN * ALIGN; }
// Every region of the weights arena and of the workspace is followed by a guard of GUARD bytes filled with
// GUARD_BYTE at pack time; no kernel may write there (dynamo_debug_check_guards counts the bytes that changed).
constexpr size_t GUARD = 256;
constexpr int GUARD_BYTE = 0xC5;

struct ArenaLayout {
    size_t header = 0;
    std::vector<size_t> w13, w2, s8m8_g, s8m8_u, mm_g, mm_u, q8_g, q8_u, cw_g, cw_u, pool_hi;
    size_t cache_idx = 0, sig_chan = 0, sig_pool = 0, sig_cnt = 0, sigmask = 0, stats = 0, stats_ctr = 0;
    size_t total = 0;
    std::vector<size_t> guards;  // offsets of the guard blocks
};

struct WsLayout {
    size_t status, counts, offsets, off_pad, topk_idx, topk_w, perm, pos, row_token, row_expert, xperm, xsig,
        hbuf, ypart,
        stage_x, stage_logits, stage_y, stage_switch, total;
    std::vector<size_t> guards;  // offsets of the guard blocks
};

inline int s_pad_of(const dynamo_layer_desc& D) { return (D.max_sig + 15) / 16 * 16; }
inline int ksplit_for(const dynamo_layer_desc& D, int T) {
    const long long R = (long long)T * (D.top_k + D.n_shared);
    return R <= DECODE_ROWS ? std::min(MAX_KSPLIT, D.d_ff / KC) : 1;
}
inline int switch_ints_per_layer(const dynamo_layer_desc& D) { return D.n_experts * (2 * s_pad_of(D) + 1); }

// Arena of the d_ff-side channel cache: header, tables, then per switchable expert the 8-bit parameters of W_down,
// the cached channels' codes, differences and bf16 originals.
struct DownLayout {
    size_t cache_idx = 0, sig_chan = 0, sig_pool = 0, sig_cnt = 0, hi_bits = 0;
    std::vector<size_t> s8m8, gminmax, q8, delta, cache_w;
    size_t total = 0;
};

void down_layout(const dynamo_layer_desc& D, const int32_t* bits, int P2, int S2, DownLayout& A) {
    const size_t d = D.d_model, f = D.d_ff, G = D.group_size, E = D.n_experts;
    size_t off = align_up(sizeof(DownDev));
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    A.cache_idx = take(E * P2 * 4);
    A.sig_chan = take(E * (size_t)std::max(S2, 1) * 4);
    A.sig_pool = take(E * (size_t)std::max(S2, 1) * 4);
    A.sig_cnt = take(E * 4);
    A.hi_bits = take(E * 4);
    A.s8m8.assign(E, 0); A.gminmax.assign(E, 0); A.q8.assign(E, 0); A.delta.assign(E, 0); A.cache_w.assign(E, 0);
    for (size_t e = 0; e < E; ++e) {
        if (bits[e] >= HI_BITS) continue;
        A.s8m8[e] = take(d * (f / G) * 4);
        A.gminmax[e] = take(d * (f / G) * 4);
        A.q8[e] = take((size_t)P2 * d);
        A.delta[e] = take((size_t)P2 * d * 2);
        A.cache_w[e] = take((size_t)P2 * d * 2);
    }
    A.total = off;
}

dynamo_status check_down_sizes(const dynamo_layer_desc& D, int P2, int S2) {
    if (P2 < 1 || P2 > D.d_ff || P2 > 65535 || S2 < 0 || S2 > 256 || S2 > P2) return DYNAMO_ERR_SHAPE;
    return DYNAMO_OK;
}

dynamo_status check_desc(const dynamo_layer_desc* D) {
    if (!D) return DYNAMO_ERR_NULL;
    if (D->d_model <= 0 || D->d_ff <= 0 || D->d_model % 256 || D->d_ff % 128) return DYNAMO_ERR_SHAPE;
    if (D->group_size != 64 && D->group_size != 128) return DYNAMO_ERR_SHAPE;
    if (D->n_experts < 1 || D->n_experts > 256 || D->n_shared < 0 || D->n_experts + D->n_shared > MAX_EXPERTS)
        return DYNAMO_ERR_SHAPE;
    if (D->top_k < 1 || D->top_k > 8 || D->top_k > D->n_experts) return DYNAMO_ERR_SHAPE;
    if (D->max_sig < 0 || D->max_sig > 256 || D->cache_size < D->max_sig || D->cache_size > D->d_model ||
        D->cache_size > 65535)
        return DYNAMO_ERR_SHAPE;
    if (D->max_tokens < 1 || (long long)D->max_tokens * (D->top_k + D->n_shared) > (1ll << 24)) return DYNAMO_ERR_SHAPE;
    return DYNAMO_OK;
}

dynamo_status check_bits(const dynamo_layer_desc& D, const int32_t* bits) {
    if (!bits) return DYNAMO_ERR_NULL;
    for (int e = 0; e < D.n_experts + D.n_shared; ++e) {
        const int b = bits[e];
        if (e >= D.n_experts) {
            if (b != 8) return DYNAMO_ERR_BITS;
        } else if (b != 2 && b != 3 && b != 4 && b != 6 && b != 8) {
            return DYNAMO_ERR_BITS;
        }
    }
    return DYNAMO_OK;
}

void arena_layout(const dynamo_layer_desc& D, const int32_t* bits, ArenaLayout& A) {
    const int n = D.n_experts + D.n_shared;
    const size_t d = D.d_model, f = D.d_ff, G = D.group_size, P = D.cache_size;
    const size_t n_rb13 = 2 * f / RB, n_kc13 = d / KC, n_rb2 = d / RB, n_kc2 = f / KC;
    A.guards.clear();
    size_t off = 0;
    A.header = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off = align_up(off + bytes);
        A.guards.push_back(off);
        off += GUARD;
        return o;
    };
    take(sizeof(LayerDev));
    A.w13.assign(n, 0); A.w2.assign(n, 0);
    A.s8m8_g.assign(n, 0); A.s8m8_u.assign(n, 0); A.q8_g.assign(n, 0); A.q8_u.assign(n, 0);
    A.mm_g.assign(n, 0); A.mm_u.assign(n, 0);
    A.cw_g.assign(n, 0); A.cw_u.assign(n, 0); A.pool_hi.assign(n, 0);
    for (int e = 0; e < n; ++e) {
        const size_t blk = block_bytes(bits[e], (int)G);
        A.w13[e] = take(n_rb13 * n_kc13 * blk);
        A.w2[e] = take(n_rb2 * n_kc2 * blk);
    }
    for (int e = 0; e < D.n_experts; ++e) {
        if (bits[e] >= HI_BITS) continue;
        A.s8m8_g[e] = take(f * (d / G) * 4);
        A.s8m8_u[e] = take(f * (d / G) * 4);
        A.mm_g[e] = take(f * (d / G) * 4);
        A.mm_u[e] = take(f * (d / G) * 4);
        A.q8_g[e] = take(P * f);
        A.q8_u[e] = take(P * f);
        A.cw_g[e] = take(P * f * 2);
        A.cw_u[e] = take(P * f * 2);
        A.pool_hi[e] = take(n_rb13 * ((P + 31) / 32 * 32) * POOL_TILE_PITCH);
    }
    const size_t S_pad = s_pad_of(D);
    A.cache_idx = take((size_t)D.n_experts * P * 4);
    A.sig_chan = take((size_t)D.n_experts * S_pad * 4);
    A.sig_pool = take((size_t)D.n_experts * S_pad * 4);
    A.sig_cnt = take((size_t)D.n_experts * 4);
    A.sigmask = take((size_t)D.n_experts * (d / 32) * 4);
    A.stats = take((size_t)D.n_experts * ((P + 31) / 32 * 32) * 4);  // activation mass per (expert, cached channel)
    A.stats_ctr = take((size_t)D.n_experts * 4);                     // arrival counters of the statistics kernel's slices
    A.total = off;
}

void ws_layout(const dynamo_layer_desc& D, WsLayout& W) {
    const size_t n = D.n_experts + D.n_shared, T = D.max_tokens, k = D.top_k, kk = D.top_k + D.n_shared;
    const size_t R = T * kk, d = D.d_model, f = D.d_ff, S_pad = s_pad_of(D);
    size_t off = 0;
    W.guards.clear();
    auto take = [&](size_t bytes) {
        size_t o = off;
        off = align_up(off + bytes);
        W.guards.push_back(off);
        off += GUARD;
        return o;
    };
    W.status = take(256);
    W.counts = take(n * 4);
    W.offsets = take((n + 1) * 4);
    W.off_pad = take((n + 1) * 4);
    W.topk_idx = take(T * k * 4);
    W.topk_w = take(T * k * 4);
    W.perm = take(T * k * 4);
    W.pos = take(T * kk * 4);
    const size_t Rp = R + 8 * n;  // physical rows: every expert's segment starts at a multiple of 8
    W.row_token = take(Rp * 4);
    W.row_expert = take(Rp * 4);
    W.xperm = take((Rp + ROW_PAD) * (d / KC) * XROW);
    W.xsig = take((Rp + ROW_PAD) * std::max<size_t>(((size_t)D.cache_size + 31) / 32 * 32, 32) * 2);  // pool columns
    W.hbuf = take((Rp + ROW_PAD) * (f / KC) * XROW);
    const size_t ks = std::min<size_t>(MAX_KSPLIT, f / KC);
    const size_t small_rows = std::min<size_t>(R, DECODE_ROWS);
    W.ypart = take(std::max(Rp, ks * (small_rows + 8 * n)) * d * 4);   // fp32 rows of the down GEMM, per K split
    W.stage_x = take(T * d * 2);
    W.stage_logits = take(T * (size_t)D.n_experts * 4);
    W.stage_y = take(T * d * 4);
    W.stage_switch = take((size_t)MAX_SWITCH_LAYERS * (switch_ints_per_layer(D) + (size_t)D.n_experts * S_pad) * 4);
    W.total = off;
}

}  // namespace

struct dynamo_ctx {
    dynamo_layer_desc D;
    bool packed = false;
    std::vector<int32_t> bits;
    std::vector<int32_t> hi_bits;                // precision the significant channels of each routed expert are served at
    // d_ff-side channel cache (optional, its own caller-owned arena)
    uint8_t* down_arena = nullptr;
    int P2 = 0, S2 = 0;
    DownLayout DA;
    std::vector<int32_t> cache_idx_down;         // host copy [E][P2]
    std::vector<std::vector<int32_t>> sig_down;  // current sets, in slot order
    std::vector<int32_t> hi_bits_down;           // precision the significant hidden units of each routed expert are served at
    std::vector<uint8_t> down_hdr;               // host copy of the d_ff-side cache's device header
    int down_active = 0;                         // experts whose d_ff-side set is not empty
    std::vector<int32_t> cache_idx;              // host copy [E][P]
    std::vector<std::vector<int32_t>> sig;       // current sets, in slot order
    ArenaLayout A;
    WsLayout W;
    uint8_t* arena = nullptr;
    uint8_t* ws = nullptr;
    LayerDev host_layer;                         // host mirror of the arena header
    int switch_mode = DYNAMO_SWITCH_SELECT;
    int tc_min_rows = TC_MIN_ROWS;               // experts with more rows take the tcgen05 path
    int operand_dtype = DYNAMO_OPERAND_FP16;     // precision the hidden activations carry into the down GEMM
    int collect_stats = 0;                       // 1: every forward adds to the per-channel activation statistics
    int n_sms = 148;                             // SM count of the device the layer was packed on
    int tc2_clusters[2] = {0, 0};                // resident CTA pairs of the tcgen05 kernel there (down, gate/up)
    int64_t launches = 0;
    cudaEvent_t prof_ev[3] = {nullptr, nullptr, nullptr};  // optional: before gate/up, after gate/up, after down
    std::vector<int32_t> upload;                 // scratch for switch uploads
    // Sets chosen on the device (dynamo_select_significant) come back through a pinned buffer and an event; the host
    // mirror `sig` is brought up to date by the next call that reads it.
    int32_t* mirror_host = nullptr;              // pinned [E][S_pad]
    cudaEvent_t mirror_ev = nullptr;
    bool mirror_pending = false;
    ~dynamo_ctx() {
        if (mirror_ev) {
            cudaEventSynchronize(mirror_ev);
            cudaEventDestroy(mirror_ev);
        }
        if (mirror_host) cudaFreeHost(mirror_host);
    }
};

namespace {

WsDev make_ws(const dynamo_ctx* c, int T) {
    const dynamo_layer_desc& D = c->D;
    WsDev w;
    uint8_t* b = c->ws;
    w.counts = (int32_t*)(b + c->W.counts);
    w.offsets = (int32_t*)(b + c->W.offsets);
    w.topk_idx = (int32_t*)(b + c->W.topk_idx);
    w.topk_w = (float*)(b + c->W.topk_w);
    w.perm = (int32_t*)(b + c->W.perm);
    w.pos = (int32_t*)(b + c->W.pos);
    w.row_token = (int32_t*)(b + c->W.row_token);
    w.row_expert = (int32_t*)(b + c->W.row_expert);
    w.xperm = b + c->W.xperm;
    w.xsig = (__half*)(b + c->W.xsig);
    w.hbuf = b + c->W.hbuf;
    w.ypart = (float*)(b + c->W.ypart);
    w.status = (int32_t*)(b + c->W.status);
    w.T = T;
    w.R = T * (D.top_k + D.n_shared);
    w.ksplit = ksplit_for(D, T);
    w.off_pad = (int32_t*)(b + c->W.off_pad);
    w.Rpad = w.R + 8 * (D.n_experts + D.n_shared);
    w.Rcap = D.max_tokens * (D.top_k + D.n_shared) + 8 * (D.n_experts + D.n_shared) + ROW_PAD;
    // No expert can exceed T rows.  Up to twice the threshold the streaming kernel takes a large expert as
    // chunks of 24 tokens (the later passes over its blocks hit L2), which costs less than two more launches.
    w.tc_min = (c->tc_min_rows != 0x7fffffff && T > 2 * c->tc_min_rows) ? c->tc_min_rows : 0x7fffffff;
    w.h_bf16 = c->operand_dtype == DYNAMO_OPERAND_BF16;
    return w;
}

#define CUDA_TRY(expr)                                  \
    do {                                                \
        cudaError_t err__ = (expr);                     \
        if (err__ != cudaSuccess) return DYNAMO_ERR_CUDA; \
    } while (0)

// Validate one layer's new sets against its cache; on success fill `lists` (slot order = caller order).
dynamo_status validate_sets(const dynamo_ctx* c, const int32_t* sig_idx, const int32_t* sig_cnt,
                            std::vector<std::vector<int32_t>>& lists) {
    const dynamo_layer_desc& D = c->D;
    lists.assign(D.n_experts, {});
    std::vector<uint8_t> seen(D.d_model);
    for (int e = 0; e < D.n_experts; ++e) {
        const int cnt = sig_cnt[e];
        if (cnt < 0 || cnt > D.max_sig) return DYNAMO_ERR_INDEX_RANGE;
        std::fill(seen.begin(), seen.end(), 0);
        const int32_t* ci = c->cache_idx.data() + (size_t)e * D.cache_size;
        for (int j = 0; j < cnt; ++j) {
            const int ch = sig_idx[(size_t)e * D.max_sig + j];
            if (ch < 0 || ch >= D.d_model) return DYNAMO_ERR_INDEX_RANGE;
            if (seen[ch]) return DYNAMO_ERR_INDEX_DUP;
            seen[ch] = 1;
            if (!std::binary_search(ci, ci + D.cache_size, ch)) return DYNAMO_ERR_NOT_CACHED;
            lists[e].push_back(ch);
        }
    }
    return DYNAMO_OK;
}

}  // namespace

extern "C" {

const char* dynamo_status_str(dynamo_status s) {
    switch (s) {
        case DYNAMO_OK: return "ok";
        case DYNAMO_ERR_NULL: return "null pointer";
        case DYNAMO_ERR_SHAPE: return "unsupported shape";
        case DYNAMO_ERR_BITS: return "unsupported bit-width";
        case DYNAMO_ERR_ALIGN: return "buffer not 256-byte aligned";
        case DYNAMO_ERR_ARENA_TOO_SMALL: return "arena or workspace too small";
        case DYNAMO_ERR_INDEX_RANGE: return "channel index or count out of range";
        case DYNAMO_ERR_INDEX_DUP: return "duplicate or unsorted channel index";
        case DYNAMO_ERR_NOT_CACHED: return "channel not in the expert's channel cache";
        case DYNAMO_ERR_STATE: return "experts not packed yet";
        case DYNAMO_ERR_TOKENS: return "token count out of range";
        case DYNAMO_ERR_CUDA: return "CUDA runtime error";
        case DYNAMO_ERR_TIMEOUT: return "device-side wait expired";
        case DYNAMO_ERR_ARG: return "argument value outside its domain";
        case DYNAMO_ERR_RANGE: return "an activation was clamped to the fp16 operand range";
    }
    return "unknown status";
}

dynamo_status dynamo_create(const dynamo_layer_desc* desc, dynamo_ctx** out) {
    if (!out) return DYNAMO_ERR_NULL;
    *out = nullptr;
    dynamo_status st = check_desc(desc);
    if (st != DYNAMO_OK) return st;
    dynamo_ctx* c = new (std::nothrow) dynamo_ctx();
    if (!c) return DYNAMO_ERR_NULL;
    c->D = *desc;
    c->D.renormalize = desc->renormalize ? 1 : 0;
    ws_layout(c->D, c->W);
    *out = c;
    return DYNAMO_OK;
}

dynamo_status dynamo_destroy(dynamo_ctx* ctx) {
    if (!ctx) return DYNAMO_ERR_NULL;
    delete ctx;
    return DYNAMO_OK;
}

dynamo_status dynamo_arena_bytes(const dynamo_layer_desc* desc, const int32_t* bits, size_t* weights_bytes,
                                 size_t* workspace_bytes) {
    dynamo_status st = check_desc(desc);
    if (st != DYNAMO_OK) return st;
    if (!weights_bytes || !workspace_bytes) return DYNAMO_ERR_NULL;
    st = check_bits(*desc, bits);
    if (st != DYNAMO_OK) return st;
    ArenaLayout A;
    arena_layout(*desc, bits, A);
    WsLayout W;
    ws_layout(*desc, W);
    *weights_bytes = A.total;
    *workspace_bytes = W.total;
    return DYNAMO_OK;
}

int64_t dynamo_kernel_launches(const dynamo_ctx* ctx) { return ctx ? ctx->launches : 0; }

dynamo_status dynamo_set_profile_events(dynamo_ctx* ctx, void* before_gateup, void* after_gateup, void* after_down) {
    if (!ctx) return DYNAMO_ERR_NULL;
    ctx->prof_ev[0] = (cudaEvent_t)before_gateup;
    ctx->prof_ev[1] = (cudaEvent_t)after_gateup;
    ctx->prof_ev[2] = (cudaEvent_t)after_down;
    return DYNAMO_OK;
}

dynamo_status dynamo_set_operand_dtype(dynamo_ctx* ctx, int32_t operand_dtype) {
    if (!ctx) return DYNAMO_ERR_NULL;
    if (operand_dtype != DYNAMO_OPERAND_FP16 && operand_dtype != DYNAMO_OPERAND_BF16) return DYNAMO_ERR_ARG;
    ctx->operand_dtype = operand_dtype;
    return DYNAMO_OK;
}

dynamo_status dynamo_set_tc_min_rows(dynamo_ctx* ctx, int32_t rows) {
    if (!ctx) return DYNAMO_ERR_NULL;
    if (rows < 0) return DYNAMO_ERR_SHAPE;
    // the streaming path handles at most 32 rows (two chunks) per expert when both paths are active
    ctx->tc_min_rows = rows == 0 ? 0x7fffffff : (rows < TC_MIN_ROWS ? rows : TC_MIN_ROWS);
    return DYNAMO_OK;
}

dynamo_status dynamo_set_channel_precision(dynamo_ctx* ctx, const int32_t* hi_bits, void* stream) {
    if (!ctx || !hi_bits) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    const dynamo_layer_desc& D = ctx->D;
    for (int e = 0; e < D.n_experts; ++e) {
        const int b = hi_bits[e];
        if (b != 2 && b != 3 && b != 4 && b != 6 && b != 8) return DYNAMO_ERR_BITS;  // nothing changes on an error
    }
    cudaStream_t st = (cudaStream_t)stream;
    for (int e = 0; e < D.n_experts; ++e) {
        if (ctx->bits[e] >= HI_BITS || ctx->hi_bits[e] == hi_bits[e]) continue;  // 8-bit experts have no cache pool
        CUDA_TRY(launch_retarget((LayerDev*)ctx->arena, e, D.d_ff, hi_bits[e], st));
        ctx->hi_bits[e] = hi_bits[e];
        ctx->host_layer.ex[e].hi_bits = hi_bits[e];
        ctx->launches += 1;
    }
    return DYNAMO_OK;
}

// Wait for the sets the device chose last (if any are still on their way) and update the host mirror.
static dynamo_status sync_mirror(dynamo_ctx* ctx) {
    if (!ctx->mirror_pending) return DYNAMO_OK;
    CUDA_TRY(cudaEventSynchronize(ctx->mirror_ev));
    const int E = ctx->D.n_experts, S_pad = s_pad_of(ctx->D);
    for (int e = 0; e < E; ++e) {
        std::vector<int32_t>& lst = ctx->sig[e];
        lst.clear();
        for (int j = 0; j < S_pad && ctx->mirror_host[(size_t)e * S_pad + j] >= 0; ++j)
            lst.push_back(ctx->mirror_host[(size_t)e * S_pad + j]);
    }
    ctx->mirror_pending = false;
    return DYNAMO_OK;
}

dynamo_status dynamo_sync_sets(dynamo_ctx* ctx, int32_t* sig_idx_out, int32_t* sig_cnt_out) {
    if (!ctx) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    dynamo_status s = sync_mirror(ctx);
    if (s != DYNAMO_OK) return s;
    const dynamo_layer_desc& D = ctx->D;
    for (int e = 0; e < D.n_experts; ++e) {
        const std::vector<int32_t>& lst = ctx->sig[e];
        if (sig_cnt_out) sig_cnt_out[e] = (int32_t)lst.size();
        if (sig_idx_out)
            for (int j = 0; j < D.max_sig; ++j) sig_idx_out[(size_t)e * D.max_sig + j] = j < (int)lst.size() ? lst[j] : -1;
    }
    return DYNAMO_OK;
}

dynamo_status dynamo_set_stats_collection(dynamo_ctx* ctx, int32_t on) {
    if (!ctx) return DYNAMO_ERR_NULL;
    ctx->collect_stats = on ? 1 : 0;
    return DYNAMO_OK;
}

dynamo_status dynamo_get_channel_stats(dynamo_ctx* ctx, float* stats_out, void* stream) {
    if (!ctx || !stats_out) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    const dynamo_layer_desc& D = ctx->D;
    const size_t P = D.cache_size, P_pad = (P + 31) / 32 * 32;
    CUDA_TRY(cudaMemcpy2DAsync(stats_out, P * 4, ctx->arena + ctx->A.stats, P_pad * 4, P * 4, D.n_experts,
                               cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return DYNAMO_OK;
}

dynamo_status dynamo_select_significant(dynamo_ctx* ctx, int32_t n_select, int32_t reset, int32_t* sig_idx_out,
                                        int32_t* sig_cnt_out, void* stream) {
    if (!ctx) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    const dynamo_layer_desc& D = ctx->D;
    if (n_select < 0 || n_select > D.max_sig) return DYNAMO_ERR_SHAPE;
    if ((size_t)D.cache_size * 4 > 48 * 1024) return DYNAMO_ERR_SHAPE;  // the ranking keeps a pool's statistics in shared memory
    cudaStream_t st = (cudaStream_t)stream;
    const int E = D.n_experts, S_pad = s_pad_of(D);
    dynamo_status ms = sync_mirror(ctx);   // the pinned buffer is about to be reused
    if (ms != DYNAMO_OK) return ms;
    if (!ctx->mirror_host) {
        CUDA_TRY(cudaMallocHost((void**)&ctx->mirror_host, (size_t)E * S_pad * 4));
        CUDA_TRY(cudaEventCreateWithFlags(&ctx->mirror_ev, cudaEventDisableTiming));
    }
    int32_t* chosen = (int32_t*)(ctx->ws + ctx->W.stage_switch);
    CUDA_TRY(launch_select((const LayerDev*)ctx->arena, (float*)(ctx->arena + ctx->A.stats), E, D.cache_size, n_select,
                           reset ? 1 : 0, chosen, st));
    ctx->launches += 1;
    // the host mirror of the sets (stream bytes, later switches in requantize mode) follows the device's choice: the
    // chosen sets travel to a pinned buffer in stream order and are read when the host next needs them
    CUDA_TRY(cudaMemcpyAsync(ctx->mirror_host, chosen, (size_t)E * S_pad * 4, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaEventRecord(ctx->mirror_ev, st));
    ctx->mirror_pending = true;
    if (sig_idx_out || sig_cnt_out) return dynamo_sync_sets(ctx, sig_idx_out, sig_cnt_out);
    return DYNAMO_OK;
}

dynamo_status dynamo_set_switch_mode(dynamo_ctx* ctx, int32_t mode) {
    if (!ctx) return DYNAMO_ERR_NULL;
    if (mode != DYNAMO_SWITCH_SELECT && mode != DYNAMO_SWITCH_REQUANT) return DYNAMO_ERR_SHAPE;
    ctx->switch_mode = mode;
    return DYNAMO_OK;
}

dynamo_status dynamo_pack_experts(dynamo_ctx* ctx, const void* w_gate, const void* w_up, const void* w_down,
                                  const int32_t* bits, const int32_t* cache_idx, void* weights_arena,
                                  size_t weights_bytes, void* workspace, size_t workspace_bytes, void* stream) {
    if (!ctx || !w_gate || !w_up || !w_down || !bits || !weights_arena || !workspace) return DYNAMO_ERR_NULL;
    const dynamo_layer_desc& D = ctx->D;
    if (D.cache_size > 0 && !cache_idx) return DYNAMO_ERR_NULL;
    dynamo_status stt = check_bits(D, bits);
    if (stt != DYNAMO_OK) return stt;
    for (int e = 0; e < D.n_experts; ++e)
        for (int p = 0; p < D.cache_size; ++p) {
            const int c = cache_idx[(size_t)e * D.cache_size + p];
            if (c < 0 || c >= D.d_model) return DYNAMO_ERR_INDEX_RANGE;
            if (p > 0 && c <= cache_idx[(size_t)e * D.cache_size + p - 1]) return DYNAMO_ERR_INDEX_DUP;
        }
    if (((uintptr_t)weights_arena % ALIGN) || ((uintptr_t)workspace % ALIGN)) return DYNAMO_ERR_ALIGN;
    ArenaLayout A;
    arena_layout(D, bits, A);
    if (weights_bytes < A.total || workspace_bytes < ctx->W.total) return DYNAMO_ERR_ARENA_TOO_SMALL;

    cudaStream_t st = (cudaStream_t)stream;
    const int n = D.n_experts + D.n_shared;
    const int d = D.d_model, f = D.d_ff, G = D.group_size, P = D.cache_size;
    ctx->packed = false;
    ctx->A = A;
    ctx->arena = (uint8_t*)weights_arena;
    ctx->ws = (uint8_t*)workspace;
    ctx->bits.assign(bits, bits + n);
    ctx->hi_bits.assign(D.n_experts, HI_BITS);
    ctx->down_arena = nullptr;  // a d_ff-side cache belongs to the previous packing
    ctx->down_active = 0;
    ctx->cache_idx.assign(cache_idx, cache_idx + (size_t)D.n_experts * P);
    if (ctx->mirror_pending) {  // sets chosen for the previous packing: let the copy land, then drop them
        CUDA_TRY(cudaEventSynchronize(ctx->mirror_ev));
        ctx->mirror_pending = false;
    }
    ctx->sig.assign(D.n_experts, {});

    CUDA_TRY(cudaMemsetAsync(ctx->arena, 0, A.total, st));
    CUDA_TRY(cudaMemsetAsync(ctx->ws, 0, ctx->W.total, st));
    for (size_t g : A.guards) CUDA_TRY(cudaMemsetAsync(ctx->arena + g, GUARD_BYTE, GUARD, st));
    for (size_t g : ctx->W.guards) CUDA_TRY(cudaMemsetAsync(ctx->ws + g, GUARD_BYTE, GUARD, st));

    LayerDev& L = ctx->host_layer;
    std::memset(&L, 0, sizeof(L));
    L.d = d; L.f = f; L.E = D.n_experts; L.Es = D.n_shared; L.k = D.top_k; L.G = G;
    L.S = D.max_sig; L.S_pad = s_pad_of(D); L.P = P; L.renorm = D.renormalize;
    L.P_pad = (P + 31) / 32 * 32;
    L.n_rb13 = 2 * f / RB; L.n_kc13 = d / KC; L.n_rb2 = d / RB; L.n_kc2 = f / KC;
    uint8_t* base = ctx->arena;
    L.cache_idx = (int32_t*)(base + A.cache_idx);
    L.sig_chan = (int32_t*)(base + A.sig_chan);
    L.sig_pool = (int32_t*)(base + A.sig_pool);
    L.sig_cnt = (int32_t*)(base + A.sig_cnt);
    L.sigmask = (uint32_t*)(base + A.sigmask);
    std::vector<int> order(n);
    for (int e = 0; e < n; ++e) order[e] = e;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return bits[a] > bits[b]; });
    for (int e = 0; e < n; ++e) L.order[e] = order[e];
    for (int e = 0; e < n; ++e) {
        ExpertDev& x = L.ex[e];
        x.bits = bits[e];
        x.blk_bytes = block_bytes(bits[e], G);
        x.w13 = base + A.w13[e];
        x.w2 = base + A.w2[e];
        x.switchable = (e < D.n_experts && bits[e] < HI_BITS) ? 1 : 0;
        x.hi_bits = HI_BITS;
        if (x.switchable) {
            x.s8m8[0] = (uint32_t*)(base + A.s8m8_g[e]);
            x.s8m8[1] = (uint32_t*)(base + A.s8m8_u[e]);
            x.gminmax[0] = (uint32_t*)(base + A.mm_g[e]);
            x.gminmax[1] = (uint32_t*)(base + A.mm_u[e]);
            x.pool_q8[0] = base + A.q8_g[e];
            x.pool_q8[1] = base + A.q8_u[e];
            x.cache_w[0] = (__nv_bfloat16*)(base + A.cw_g[e]);
            x.cache_w[1] = (__nv_bfloat16*)(base + A.cw_u[e]);
            x.pool_hi = (__half*)(base + A.pool_hi[e]);
        }
    }
    CUDA_TRY(cudaMemcpyAsync(base, &L, sizeof(L), cudaMemcpyHostToDevice, st));
    if (P > 0)
        CUDA_TRY(cudaMemcpyAsync(L.cache_idx, ctx->cache_idx.data(), ctx->cache_idx.size() * 4, cudaMemcpyHostToDevice,
                                 st));

    const __nv_bfloat16* wg = (const __nv_bfloat16*)w_gate;
    const __nv_bfloat16* wu = (const __nv_bfloat16*)w_up;
    const __nv_bfloat16* wd = (const __nv_bfloat16*)w_down;
    for (int e = 0; e < n; ++e) {
        const size_t eo = (size_t)e * f * d;
        CUDA_TRY(launch_pack_blocks(wg + eo, wu + eo, L.n_rb13, d, G, bits[e], 1, (void*)L.ex[e].w13, st));
        CUDA_TRY(launch_pack_blocks(wd + eo, nullptr, L.n_rb2, f, G, bits[e], 0, (void*)L.ex[e].w2, st));
        ctx->launches += 2;
        if (L.ex[e].switchable && P > 0) {
            CUDA_TRY(launch_pack_hi(wg + eo, wu + eo, f, d, G, P, L.cache_idx + (size_t)e * P, L.ex[e], st));
            ctx->launches += 1;
        }
    }
    {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
            ctx->n_sms = sms;
        CUDA_TRY(setup_ffn_tc2(ctx->n_sms, ctx->tc2_clusters));
    }
    ctx->packed = true;
    // install the empty significant sets (sig_pool -> zero tile, sig_chan -> -1)
    std::vector<int32_t> zero_cnt(D.n_experts, 0);
    std::vector<int32_t> dummy((size_t)D.n_experts * std::max(1, D.max_sig), 0);
    dynamo_status s2 = dynamo_set_channel_switch(ctx, dummy.data(), zero_cnt.data(), stream);
    if (s2 != DYNAMO_OK) ctx->packed = false;
    return s2;
}

dynamo_status dynamo_set_channel_switch_many(dynamo_ctx* const* ctxs, int32_t n_layers, const int32_t* sig_idx,
                                             const int32_t* sig_cnt, void* stream) {
    if (!ctxs || !sig_idx || !sig_cnt) return DYNAMO_ERR_NULL;
    if (n_layers < 1 || n_layers > MAX_SWITCH_LAYERS) return DYNAMO_ERR_SHAPE;
    for (int l = 0; l < n_layers; ++l) {
        if (!ctxs[l]) return DYNAMO_ERR_NULL;
        if (!ctxs[l]->packed) return DYNAMO_ERR_STATE;
        if (std::memcmp(&ctxs[l]->D, &ctxs[0]->D, sizeof(dynamo_layer_desc)) != 0) return DYNAMO_ERR_SHAPE;
    }
    for (int l = 0; l < n_layers; ++l) {  // sets the device chose earlier enter the host mirror first
        dynamo_status ms = sync_mirror(ctxs[l]);
        if (ms != DYNAMO_OK) return ms;
    }
    dynamo_ctx* c0 = ctxs[0];
    const dynamo_layer_desc& D = c0->D;
    const int E = D.n_experts, S = D.max_sig, S_pad = s_pad_of(D), P = D.cache_size;
    const int per_layer = switch_ints_per_layer(D);
    // validate everything first: all-or-nothing
    std::vector<std::vector<std::vector<int32_t>>> lists(n_layers);
    for (int l = 0; l < n_layers; ++l) {
        dynamo_status st = validate_sets(ctxs[l], sig_idx + (size_t)l * E * S, sig_cnt + (size_t)l * E, lists[l]);
        if (st != DYNAMO_OK) return st;
    }
    cudaStream_t st = (cudaStream_t)stream;
    std::vector<int32_t>& up = c0->upload;
    up.assign((size_t)n_layers * per_layer, 0);
    SwitchLayers layers;
    std::memset(&layers, 0, sizeof(layers));
    int32_t* staging = (int32_t*)(c0->ws + c0->W.stage_switch);
    int32_t* items_dev = staging + (size_t)MAX_SWITCH_LAYERS * per_layer;
    for (int l = 0; l < n_layers; ++l) {
        dynamo_ctx* c = ctxs[l];
        layers.layer[l] = (const LayerDev*)c->arena;
        int32_t* chan = up.data() + (size_t)l * per_layer;
        int32_t* pool = chan + (size_t)E * S_pad;
        int32_t* cnt = pool + (size_t)E * S_pad;
        std::vector<int32_t> items;  // entering cached channels (expert << 16 | pool position)
        for (int e = 0; e < E; ++e) {
            const int32_t* ci = c->cache_idx.data() + (size_t)e * P;
            const bool sw = c->bits[e] < HI_BITS;
            const std::vector<int32_t>& lst = lists[l][e];
            cnt[e] = sw ? (int32_t)lst.size() : 0;
            for (int j = 0; j < S_pad; ++j) {
                chan[e * S_pad + j] = -1;
                pool[e * S_pad + j] = P;
            }
            if (!sw) continue;
            for (size_t j = 0; j < lst.size(); ++j) {
                const int p = (int)(std::lower_bound(ci, ci + P, lst[j]) - ci);
                chan[e * S_pad + j] = lst[j];
                pool[e * S_pad + j] = p;
                if (c->switch_mode == DYNAMO_SWITCH_REQUANT &&
                    std::find(c->sig[e].begin(), c->sig[e].end(), lst[j]) == c->sig[e].end())
                    items.push_back((e << 16) | p);
            }
        }
        if (!items.empty()) {
            // channel replacement + requantization of the entering channels from the bf16 cache
            int32_t* dst = items_dev + (size_t)l * E * S_pad;
            CUDA_TRY(cudaMemcpyAsync(dst, items.data(), items.size() * 4, cudaMemcpyHostToDevice, st));
            CUDA_TRY(launch_requant(layers.layer[l], D.d_ff, dst, (int)items.size(), st));
            c->launches += 1;
        }
    }
    CUDA_TRY(cudaMemcpyAsync(staging, up.data(), up.size() * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(launch_switch(layers, n_layers, E, staging, per_layer, st));
    c0->launches += 1;
    for (int l = 0; l < n_layers; ++l) ctxs[l]->sig = lists[l];
    return DYNAMO_OK;
}

dynamo_status dynamo_set_channel_switch(dynamo_ctx* ctx, const int32_t* sig_idx, const int32_t* sig_cnt,
                                        void* stream) {
    if (!ctx) return DYNAMO_ERR_NULL;
    dynamo_ctx* one[1] = {ctx};
    return dynamo_set_channel_switch_many(one, 1, sig_idx, sig_cnt, stream);
}

// Optional copies of the routing intermediates for parity tests.
static dynamo_status forward_debug_copies(const dynamo_ctx* ctx, const WsDev& ws, int32_t T, const dynamo_debug_out* dbg,
                                          cudaStream_t st) {
    if (!dbg) return DYNAMO_OK;
    const dynamo_layer_desc& D = ctx->D;
    const size_t tk = (size_t)T * D.top_k;
    if (dbg->topk_idx) CUDA_TRY(cudaMemcpyAsync(dbg->topk_idx, ws.topk_idx, tk * 4, cudaMemcpyDeviceToDevice, st));
    if (dbg->topk_w) CUDA_TRY(cudaMemcpyAsync(dbg->topk_w, ws.topk_w, tk * 4, cudaMemcpyDeviceToDevice, st));
    if (dbg->expert_offsets)
        CUDA_TRY(cudaMemcpyAsync(dbg->expert_offsets, ws.offsets, (size_t)(D.n_experts + 1) * 4,
                                 cudaMemcpyDeviceToDevice, st));
    if (dbg->perm) CUDA_TRY(cudaMemcpyAsync(dbg->perm, ws.perm, tk * 4, cudaMemcpyDeviceToDevice, st));
    return DYNAMO_OK;
}

// The forward from either given router logits or the router's weights (then the scores are computed by the
// fused GEMM + top-k kernel, and written to logits_out if that is not NULL).
static dynamo_status forward_impl(dynamo_ctx* ctx, const void* x, const float* router_logits, const void* w_router,
                                  const float* router_bias, float* logits_out, int32_t T, void* y, int32_t y_dtype,
                                  const dynamo_debug_out* dbg, void* stream) {
    if (!ctx) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    const dynamo_layer_desc& D = ctx->D;
    if (T < 0 || T > D.max_tokens) return DYNAMO_ERR_TOKENS;
    if (y_dtype != DYNAMO_BF16 && y_dtype != DYNAMO_F32) return DYNAMO_ERR_SHAPE;
    if (T == 0) return DYNAMO_OK;
    if (!x || (!router_logits && !w_router) || !y) return DYNAMO_ERR_NULL;
    // 16-byte vector loads of x (and of the router weights), 16-byte vector stores of y
    if ((((uintptr_t)x | (uintptr_t)y) & 15) || (w_router && ((uintptr_t)w_router & 15))) return DYNAMO_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    const LayerDev* L = (const LayerDev*)ctx->arena;
    WsDev ws = make_ws(ctx, T);
    const int n = D.n_experts + D.n_shared;

    const bool fused_front = !w_router && front_fits(T, D.top_k);   // small batch: routing, permutation, gather in one launch
    if (fused_front) {
        CUDA_TRY(launch_front(L, ws, x, router_logits, D.n_experts, D.n_shared, D.top_k, D.renormalize, st));
    } else {
        if (w_router)
            CUDA_TRY(launch_route_gemm(x, w_router, router_bias, T, D.d_model, D.n_experts, D.top_k, D.renormalize,
                                       logits_out, ws.topk_idx, ws.topk_w, st));
        else
            CUDA_TRY(launch_route(router_logits, T, D.n_experts, D.top_k, D.renormalize, ws.topk_idx, ws.topk_w, st));
        CUDA_TRY(launch_scan(ws, D.n_experts, D.n_shared, D.top_k, st));
        CUDA_TRY(launch_gather(L, ws, x, st));
    }
    if (ctx->collect_stats) {
        // row slices per expert: about two CTAs per SM in all; the partial sums live in the down GEMM's output buffer
        // (at least 8 * (E + Es) rows of d floats, idle until the down launch), which bounds the slice count
        const int P_pad = ctx->host_layer.P_pad;
        int n_slices = std::max(1, std::min(32, (2 * ctx->n_sms + D.n_experts - 1) / D.n_experts));
        n_slices = std::max(1, std::min(n_slices, 8 * D.d_model / std::max(P_pad, 1)));
        if ((long long)T * D.top_k <= 16ll * D.n_experts) n_slices = 1;  // a few rows per expert: one pass is shorter
        CUDA_TRY(launch_stats(L, ws, x, (float*)(ctx->arena + ctx->A.stats), ws.ypart,
                              (int32_t*)(ctx->arena + ctx->A.stats_ctr), D.n_experts, n_slices, st));
        ctx->launches += 1;
    }
    const bool use_tc = ws.tc_min != 0x7fffffff;                  // experts above 32 rows take the tcgen05 path
    const long long split_stride = (long long)ws.Rpad * D.d_model;  // partials of one K split: [Rpad][d]
    if (ctx->prof_ev[0]) CUDA_TRY(cudaEventRecord(ctx->prof_ev[0], st));
    const int max_rows = use_tc ? std::min(T, ctx->tc_min_rows) : T;  // rows one expert can have on the streaming path
    CUDA_TRY(launch_ffn_stream(L, ws, 1, ctx->host_layer.n_rb13, 1, n, split_stride, max_rows, ctx->n_sms,
                               D.group_size, st));
    if (use_tc) CUDA_TRY(launch_ffn_tc2(L, ws, 1, ctx->host_layer.n_rb13, n, ctx->tc2_clusters[1], st));
    if (ctx->prof_ev[1]) CUDA_TRY(cudaEventRecord(ctx->prof_ev[1], st));
    CUDA_TRY(launch_ffn_stream(L, ws, 0, ctx->host_layer.n_rb2, ws.ksplit, n, split_stride, max_rows, ctx->n_sms,
                               D.group_size, st));
    if (use_tc) CUDA_TRY(launch_ffn_tc2(L, ws, 0, ctx->host_layer.n_rb2, n, ctx->tc2_clusters[0], st));
    if (ctx->prof_ev[2]) CUDA_TRY(cudaEventRecord(ctx->prof_ev[2], st));
    if (ctx->down_active) {  // significant hidden units: add what their 8-bit columns of W_down change
        CUDA_TRY(launch_down_fix(L, (const DownDev*)ctx->down_arena, ws, D.d_model, st));
        ctx->launches += 1;
    }
    CUDA_TRY(launch_combine(ws, D.d_model, D.top_k, D.n_shared, y, y_dtype == DYNAMO_F32, split_stride, st));
    ctx->launches += (use_tc ? 8 : 6) - (fused_front ? 2 : 0);
    return forward_debug_copies(ctx, ws, T, dbg, st);
}

dynamo_status dynamo_moe_forward(dynamo_ctx* ctx, const void* x, const float* router_logits, int32_t T, void* y,
                                 int32_t y_dtype, const dynamo_debug_out* dbg, void* stream) {
    if (ctx && ctx->packed && T > 0 && T <= ctx->D.max_tokens && !router_logits) return DYNAMO_ERR_NULL;
    return forward_impl(ctx, x, router_logits, nullptr, nullptr, nullptr, T, y, y_dtype, dbg, stream);
}

dynamo_status dynamo_moe_forward_router(dynamo_ctx* ctx, const void* x, const void* w_router, const float* router_bias,
                                        int32_t T, void* y, int32_t y_dtype, float* logits_out,
                                        const dynamo_debug_out* dbg, void* stream) {
    if (ctx && ctx->packed && T > 0 && T <= ctx->D.max_tokens && !w_router) return DYNAMO_ERR_NULL;
    return forward_impl(ctx, x, nullptr, w_router, router_bias, logits_out, T, y, y_dtype, dbg, stream);
}

dynamo_status dynamo_moe_forward_host(dynamo_ctx* ctx, const void* x_host, const float* logits_host, int32_t T,
                                      void* y_host, int32_t y_dtype, void* stream) {
    if (!ctx) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    const dynamo_layer_desc& D = ctx->D;
    if (T < 0 || T > D.max_tokens) return DYNAMO_ERR_TOKENS;
    if (y_dtype != DYNAMO_BF16 && y_dtype != DYNAMO_F32) return DYNAMO_ERR_SHAPE;
    if (T == 0) return DYNAMO_OK;
    if (!x_host || !logits_host || !y_host) return DYNAMO_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    void* xd = ctx->ws + ctx->W.stage_x;
    float* ld = (float*)(ctx->ws + ctx->W.stage_logits);
    void* yd = ctx->ws + ctx->W.stage_y;
    CUDA_TRY(cudaMemcpyAsync(xd, x_host, (size_t)T * D.d_model * 2, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(ld, logits_host, (size_t)T * D.n_experts * 4, cudaMemcpyHostToDevice, st));
    dynamo_status s = dynamo_moe_forward(ctx, xd, ld, T, yd, y_dtype, nullptr, stream);
    if (s != DYNAMO_OK) return s;
    const size_t ybytes = (size_t)T * D.d_model * (y_dtype == DYNAMO_F32 ? 4 : 2);
    CUDA_TRY(cudaMemcpyAsync(y_host, yd, ybytes, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    return DYNAMO_OK;
}

dynamo_status dynamo_down_cache_bytes(const dynamo_layer_desc* desc, const int32_t* bits, int32_t cache_size_down,
                                      int32_t max_sig_down, size_t* bytes) {
    if (!bytes) return DYNAMO_ERR_NULL;
    dynamo_status s = check_desc(desc);
    if (s != DYNAMO_OK) return s;
    s = check_bits(*desc, bits);
    if (s != DYNAMO_OK) return s;
    s = check_down_sizes(*desc, cache_size_down, max_sig_down);
    if (s != DYNAMO_OK) return s;
    DownLayout A;
    down_layout(*desc, bits, cache_size_down, max_sig_down, A);
    *bytes = A.total;
    return DYNAMO_OK;
}

dynamo_status dynamo_pack_down_cache(dynamo_ctx* ctx, const void* w_down, const int32_t* cache_idx_down,
                                     int32_t cache_size_down, int32_t max_sig_down, void* down_arena, size_t down_bytes,
                                     void* stream) {
    if (!ctx || !w_down || !cache_idx_down || !down_arena) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    const dynamo_layer_desc& D = ctx->D;
    dynamo_status s = check_down_sizes(D, cache_size_down, max_sig_down);
    if (s != DYNAMO_OK) return s;
    if ((uintptr_t)down_arena % ALIGN) return DYNAMO_ERR_ALIGN;
    const int P2 = cache_size_down, S2 = max_sig_down, E = D.n_experts;
    DownLayout A;
    down_layout(D, ctx->bits.data(), P2, S2, A);
    if (down_bytes < A.total) return DYNAMO_ERR_ARENA_TOO_SMALL;
    for (int e = 0; e < E; ++e)
        for (int j = 0; j < P2; ++j) {
            const int c = cache_idx_down[(size_t)e * P2 + j];
            if (c < 0 || c >= D.d_ff) return DYNAMO_ERR_INDEX_RANGE;
            if (j > 0 && c <= cache_idx_down[(size_t)e * P2 + j - 1]) return DYNAMO_ERR_INDEX_DUP;
        }
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* base = (uint8_t*)down_arena;
    ctx->down_arena = nullptr;  // stays off if anything below fails
    ctx->down_active = 0;
    ctx->P2 = P2;
    ctx->S2 = S2;
    ctx->DA = A;
    ctx->cache_idx_down.assign(cache_idx_down, cache_idx_down + (size_t)E * P2);
    ctx->sig_down.assign(E, {});
    ctx->hi_bits_down.assign(E, HI_BITS);

    std::vector<uint8_t> hdr(sizeof(DownDev), 0);
    DownDev& H = *reinterpret_cast<DownDev*>(hdr.data());
    H.P2 = P2;
    H.S2 = std::max(S2, 1);
    H.cache_idx = (int32_t*)(base + A.cache_idx);
    H.sig_chan = (int32_t*)(base + A.sig_chan);
    H.sig_pool = (int32_t*)(base + A.sig_pool);
    H.sig_cnt = (int32_t*)(base + A.sig_cnt);
    for (int e = 0; e < E; ++e) {
        if (ctx->bits[e] >= HI_BITS) continue;
        H.ex[e].s8m8 = (uint32_t*)(base + A.s8m8[e]);
        H.ex[e].gminmax = (uint32_t*)(base + A.gminmax[e]);
        H.ex[e].q8 = base + A.q8[e];
        H.ex[e].delta = (__half*)(base + A.delta[e]);
        H.ex[e].cache_w = (__nv_bfloat16*)(base + A.cache_w[e]);
    }
    CUDA_TRY(cudaMemcpyAsync(base, hdr.data(), sizeof(DownDev), cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(H.cache_idx, ctx->cache_idx_down.data(), (size_t)E * P2 * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemsetAsync(H.sig_chan, 0xff, (size_t)E * H.S2 * 4, st));
    CUDA_TRY(cudaMemsetAsync(H.sig_pool, 0, (size_t)E * H.S2 * 4, st));
    CUDA_TRY(cudaMemsetAsync(H.sig_cnt, 0, (size_t)E * 4, st));
    CUDA_TRY(cudaMemcpyAsync(base + A.hi_bits, ctx->hi_bits_down.data(), (size_t)E * 4, cudaMemcpyHostToDevice, st));
    const char* wd = (const char*)w_down;
    const size_t per_expert = (size_t)D.d_model * D.d_ff * 2;
    for (int e = 0; e < E; ++e) {
        if (ctx->bits[e] >= HI_BITS) continue;
        CUDA_TRY(launch_pack_down_hi(wd + e * per_expert, D.d_model, D.d_ff, D.group_size, P2,
                                     H.cache_idx + (size_t)e * P2, ctx->bits[e], H.ex[e], st));
        ctx->launches += 1;
    }
    CUDA_TRY(cudaStreamSynchronize(st));  // the host staging above may go away
    ctx->down_arena = base;
    ctx->down_hdr = hdr;
    return DYNAMO_OK;
}

dynamo_status dynamo_set_channel_precision_down(dynamo_ctx* ctx, const int32_t* hi_bits, void* stream) {
    if (!ctx || !hi_bits) return DYNAMO_ERR_NULL;
    if (!ctx->packed || !ctx->down_arena) return DYNAMO_ERR_STATE;
    const dynamo_layer_desc& D = ctx->D;
    for (int e = 0; e < D.n_experts; ++e) {
        const int b = hi_bits[e];
        if (b != 2 && b != 3 && b != 4 && b != 6 && b != 8) return DYNAMO_ERR_BITS;  // nothing changes on an error
    }
    cudaStream_t st = (cudaStream_t)stream;
    const DownDev& H = *reinterpret_cast<const DownDev*>(ctx->down_hdr.data());
    bool changed = false;
    for (int e = 0; e < D.n_experts; ++e) {
        if (ctx->bits[e] >= HI_BITS || ctx->hi_bits_down[e] == hi_bits[e]) continue;  // 8-bit experts have no cache
        CUDA_TRY(launch_retarget_down(D.d_model, D.d_ff, D.group_size, ctx->P2, H.cache_idx + (size_t)e * ctx->P2,
                                      ctx->bits[e], hi_bits[e], H.ex[e], st));
        ctx->hi_bits_down[e] = hi_bits[e];
        ctx->launches += 1;
        changed = true;
    }
    if (changed)  // (a copy from pageable memory returns once the source has been staged)
        CUDA_TRY(cudaMemcpyAsync(ctx->down_arena + ctx->DA.hi_bits, ctx->hi_bits_down.data(), (size_t)D.n_experts * 4,
                                 cudaMemcpyHostToDevice, st));
    return DYNAMO_OK;
}

dynamo_status dynamo_set_channel_switch_down(dynamo_ctx* ctx, const int32_t* sig_idx, const int32_t* sig_cnt,
                                             void* stream) {
    if (!ctx || !sig_idx || !sig_cnt) return DYNAMO_ERR_NULL;
    if (!ctx->packed || !ctx->down_arena) return DYNAMO_ERR_STATE;
    const dynamo_layer_desc& D = ctx->D;
    const int E = D.n_experts, P2 = ctx->P2, S2 = ctx->S2, S2d = std::max(S2, 1);
    std::vector<int32_t> chan((size_t)E * S2d, -1), pool((size_t)E * S2d, 0), cnts(E, 0);
    std::vector<std::vector<int32_t>> lists(E);
    std::vector<uint8_t> seen(D.d_ff);
    for (int e = 0; e < E; ++e) {
        const int cnt = sig_cnt[e];
        if (cnt < 0 || cnt > S2) return DYNAMO_ERR_INDEX_RANGE;
        std::fill(seen.begin(), seen.end(), 0);
        const int32_t* ci = ctx->cache_idx_down.data() + (size_t)e * P2;
        for (int j = 0; j < cnt; ++j) {
            const int ch = sig_idx[(size_t)e * S2 + j];
            if (ch < 0 || ch >= D.d_ff) return DYNAMO_ERR_INDEX_RANGE;
            if (seen[ch]) return DYNAMO_ERR_INDEX_DUP;
            seen[ch] = 1;
            const int32_t* it = std::lower_bound(ci, ci + P2, ch);
            if (it == ci + P2 || *it != ch) return DYNAMO_ERR_NOT_CACHED;
            if (ctx->bits[e] >= HI_BITS) continue;  // an 8-bit expert ignores its set
            chan[(size_t)e * S2d + lists[e].size()] = ch;
            pool[(size_t)e * S2d + lists[e].size()] = (int32_t)(it - ci);
            lists[e].push_back(ch);
        }
        cnts[e] = (int32_t)lists[e].size();
    }
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* base = ctx->down_arena;
    CUDA_TRY(cudaMemcpyAsync(base + ctx->DA.sig_chan, chan.data(), chan.size() * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(base + ctx->DA.sig_pool, pool.data(), pool.size() * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(base + ctx->DA.sig_cnt, cnts.data(), cnts.size() * 4, cudaMemcpyHostToDevice, st));
    // (copies from pageable memory return once the source has been staged, so the vectors may die with this call;
    // the tables change in stream order, between the forwards enqueued before and after)
    ctx->sig_down = lists;
    ctx->down_active = 0;
    for (int e = 0; e < E; ++e) ctx->down_active += cnts[e] > 0 ? 1 : 0;
    if (ctx->switch_mode == DYNAMO_SWITCH_REQUANT && ctx->down_active > 0) {
        // channel replacement + requantization: codes and differences of the new sets from the bf16 channel cache
        CUDA_TRY(launch_requant_down((const LayerDev*)ctx->arena, (const DownDev*)base,
                                     (const int32_t*)(base + ctx->DA.hi_bits), D.d_model, E, st));
        ctx->launches += 1;
    }
    return DYNAMO_OK;
}

dynamo_status dynamo_export_codes(dynamo_ctx* ctx, int32_t expert, int32_t matrix, uint8_t* q, uint16_t* scale_f16,
                                  uint16_t* zero_f16, int32_t which, void* stream) {
    if (!ctx || !q || !scale_f16 || !zero_f16) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    const dynamo_layer_desc& D = ctx->D;
    if (expert < 0 || expert >= D.n_experts + D.n_shared || matrix < 0 || matrix > 2 || which < 0 || which > 2)
        return DYNAMO_ERR_SHAPE;
    if (which != DYNAMO_CODES_BASE && !ctx->host_layer.ex[expert].switchable) return DYNAMO_ERR_BITS;
    const long long n_elems = (long long)D.d_model * D.d_ff;
    if (which != DYNAMO_CODES_BASE && matrix == DYNAMO_MAT_DOWN) {
        if (!ctx->down_arena) return DYNAMO_ERR_STATE;  // no d_ff-side cache packed
        CUDA_TRY(launch_export_down((const LayerDev*)ctx->arena, (const DownDev*)ctx->down_arena, expert, which, n_elems,
                                    q, scale_f16, zero_f16, (cudaStream_t)stream));
        ctx->launches += 1;
        return DYNAMO_OK;
    }
    CUDA_TRY(launch_export((const LayerDev*)ctx->arena, expert, matrix, which, n_elems, q, scale_f16, zero_f16,
                           (cudaStream_t)stream));
    ctx->launches += 1;
    return DYNAMO_OK;
}

dynamo_status dynamo_expert_stream_bytes(dynamo_ctx* ctx, int32_t expert, size_t* bytes) {
    if (!ctx || !bytes) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    const dynamo_layer_desc& D = ctx->D;
    if (expert < 0 || expert >= D.n_experts + D.n_shared) return DYNAMO_ERR_SHAPE;
    const size_t d = D.d_model, f = D.d_ff;
    dynamo_status ms = sync_mirror(ctx);
    if (ms != DYNAMO_OK) return ms;
    const size_t blocks = (2 * f / RB) * (d / KC) + (d / RB) * (f / KC);
    size_t b = blocks * (size_t)block_bytes(ctx->bits[expert], D.group_size);
    if (expert < D.n_experts && ctx->bits[expert] < HI_BITS) b += 2 * f * ctx->sig[expert].size() * 2;
    if (expert < D.n_experts && ctx->down_arena) b += d * ctx->sig_down[expert].size() * 2;
    *bytes = b;
    return DYNAMO_OK;
}

dynamo_status dynamo_poll_status(dynamo_ctx* ctx, void* stream) {
    if (!ctx) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t word = 0;
    CUDA_TRY(cudaMemcpyAsync(&word, ctx->ws + ctx->W.status, 4, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    if (word == STATUS_OK) return DYNAMO_OK;
    CUDA_TRY(cudaMemsetAsync(ctx->ws + ctx->W.status, 0, 4, st));
    if (word & STATUS_TIMEOUT) return DYNAMO_ERR_TIMEOUT;
    return DYNAMO_ERR_RANGE;
}

dynamo_status dynamo_debug_expire_wait(dynamo_ctx* ctx, int64_t limit_ns, void* stream) {
    if (!ctx) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    if (limit_ns < 1000 || limit_ns > 100ll * 1000 * 1000) return DYNAMO_ERR_ARG;
    CUDA_TRY(launch_expire_wait((int32_t*)(ctx->ws + ctx->W.status), (unsigned long long)limit_ns, (cudaStream_t)stream));
    ctx->launches += 1;
    return DYNAMO_OK;
}

dynamo_status dynamo_debug_check_guards(dynamo_ctx* ctx, int64_t* n_bad_bytes, void* stream) {
    if (!ctx || !n_bad_bytes) return DYNAMO_ERR_NULL;
    if (!ctx->packed) return DYNAMO_ERR_STATE;
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_TRY(cudaStreamSynchronize(st));
    int64_t bad = 0;
    std::vector<uint8_t> buf(GUARD);
    auto scan = [&](const uint8_t* base, const std::vector<size_t>& guards) -> cudaError_t {
        for (size_t g : guards) {
            cudaError_t err = cudaMemcpy(buf.data(), base + g, GUARD, cudaMemcpyDeviceToHost);
            if (err != cudaSuccess) return err;
            for (uint8_t b : buf) bad += b != (uint8_t)GUARD_BYTE;
        }
        return cudaSuccess;
    };
    CUDA_TRY(scan(ctx->arena, ctx->A.guards));
    CUDA_TRY(scan(ctx->ws, ctx->W.guards));
    *n_bad_bytes = bad;
    return DYNAMO_OK;
}

}  // extern "C"
