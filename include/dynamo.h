/*
 * dynamo.h - C-ABI of the B200-native DynaMo quantized-MoE hot path.
 *
 * One MoE layer = one context.  The layer's routed-expert SwiGLU FFN runs over
 * expert-level mixed-precision weights (each expert bit-packed at its own base
 * bit-width of 2, 3, 4, 6 or 8 bits, group-wise fp16 scale / fp16 zero) combined with the channel-level
 * dynamic switch: a runtime-selected set of significant input channels per expert
 * is served at 8-bit precision from the channel cache while the rest stay at the
 * expert's base precision.
 *
 * Conventions
 *  - Every function returns a dynamo_status (0 = OK).  No exceptions, no global state.
 *  - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host memory.
 *  - All device buffers are CALLER-OWNED.  The context owns only host metadata and
 *    pointers into the caller's arenas; the library never calls cudaMalloc.
 *  - Calls that touch the device take a cudaStream_t (passed as void*; NULL = the
 *    legacy default stream), are asynchronous and stream-ordered unless stated.
 *  - Argument errors are detected on the host BEFORE any launch and leave all state
 *    unchanged.  Device-side waits are bounded; an expired wait sets a status word
 *    that dynamo_poll_status reads.
 *  - One context per layer, externally synchronised (not thread-safe).
 *  - Shapes: d_model % 256 == 0, d_ff % 128 == 0, group_size in {64, 128},
 *    1 <= top_k <= 8, n_experts <= 256, n_experts + n_shared <= 264, top_k <= n_experts,
 *    max_sig <= cache_size <= d_model, max_sig <= 256.
 *  - MMA operand format is fp16 (codes and activations are exact in it; the hidden
 *    activation h is rounded to fp16); accumulation is fp32.  The operands carry a
 *    power-of-two pre-scale of up to 2^4, so activations must satisfy |x| <= 4080 and
 *    |h| <= 4080 (the largest bf16 / fp16 value below 65504 / 16).  A larger magnitude (an
 *    infinity included) is CLAMPED to +-4080, the forward completes with the clamped value
 *    (exactly the forward of the clamped input), and the sticky status bit
 *    behind DYNAMO_ERR_RANGE is set (read and cleared by dynamo_poll_status).  NaN inputs
 *    propagate.
 */
#ifndef DYNAMO_H_
#define DYNAMO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DYNAMO_OK = 0,
    DYNAMO_ERR_NULL = 1,            /* a required pointer is NULL */
    DYNAMO_ERR_SHAPE = 2,           /* a dimension violates the shape rules above */
    DYNAMO_ERR_BITS = 3,            /* a bit-width is not one of 2, 3, 4, 6, 8 (shared experts: 8) */
    DYNAMO_ERR_ALIGN = 4,           /* an arena is not 256-byte aligned, or x / y / w_router not 16-byte aligned */
    DYNAMO_ERR_ARENA_TOO_SMALL = 5, /* weights arena or workspace smaller than dynamo_arena_bytes says */
    DYNAMO_ERR_INDEX_RANGE = 6,     /* a channel index is outside [0, d_model) or a count outside [0, S] */
    DYNAMO_ERR_INDEX_DUP = 7,       /* a channel index appears twice / cache_idx not strictly increasing */
    DYNAMO_ERR_NOT_CACHED = 8,      /* a significant channel is not in that expert's channel cache */
    DYNAMO_ERR_STATE = 9,           /* call made before dynamo_pack_experts */
    DYNAMO_ERR_TOKENS = 10,         /* T < 0 or T > max_tokens */
    DYNAMO_ERR_CUDA = 11,           /* a CUDA runtime call failed */
    DYNAMO_ERR_TIMEOUT = 12,        /* a bounded device-side wait expired (see dynamo_poll_status) */
    DYNAMO_ERR_ARG = 13,            /* a scalar or array value is outside its domain */
    DYNAMO_ERR_RANGE = 14           /* an activation exceeded the fp16 operand range and was clamped (see Conventions) */
} dynamo_status;

typedef struct {
    int32_t d_model;     /* d: expert input / output width */
    int32_t d_ff;        /* f: expert hidden width */
    int32_t n_experts;   /* E: routed experts */
    int32_t n_shared;    /* E_s: always-on shared experts (8-bit, weight 1), may be 0 */
    int32_t top_k;       /* k */
    int32_t group_size;  /* G: quantization group along the input axis, 64 or 128 */
    int32_t max_sig;     /* S: capacity of one expert's significant-channel set */
    int32_t cache_size;  /* P: channels per expert kept in the channel cache (candidates) */
    int32_t max_tokens;  /* largest T a forward may be called with */
    int32_t renormalize; /* 1: the k routing weights are rescaled to sum to 1 */
} dynamo_layer_desc;

typedef struct dynamo_ctx dynamo_ctx;

/* Optional device outputs of a forward, for parity checks (any member may be NULL). */
typedef struct {
    int32_t* topk_idx;       /* dev int32 [T, k]   chosen experts, descending logit            */
    float*   topk_w;         /* dev fp32  [T, k]   routing weights                             */
    int32_t* expert_offsets; /* dev int32 [E + 1]  exclusive scan of per-expert pair counts    */
    int32_t* perm;           /* dev int32 [T * k]  sorted row -> t*k + j                       */
} dynamo_debug_out;

enum { DYNAMO_BF16 = 0, DYNAMO_F32 = 1 };                       /* y_dtype */
enum { DYNAMO_MAT_GATE = 0, DYNAMO_MAT_UP = 1, DYNAMO_MAT_DOWN = 2 };
enum { DYNAMO_CODES_BASE = 0,      /* base-precision codes and params of the whole matrix          */
       DYNAMO_CODES_HI_POOL = 1,   /* 8-bit codes of the cached channels (0 elsewhere), 8-bit params */
       DYNAMO_CODES_HI_ACTIVE = 2  /* as HI_POOL but only the currently significant channels        */ };
enum { DYNAMO_SWITCH_SELECT = 0,   /* switch = re-point the active list at codes quantized at pack time */
       DYNAMO_SWITCH_REQUANT = 1   /* switch also re-derives the entering channels' 8-bit codes from the
                                      bf16 originals in the channel cache (the paper's replace-then-requantize) */ };

/* Create / destroy a layer context.  Host only; needs no GPU.  [layer shape: Section II-A] */
dynamo_status dynamo_create(const dynamo_layer_desc* desc, dynamo_ctx** out);
dynamo_status dynamo_destroy(dynamo_ctx* ctx);

/* (Utility call: the paper has no counterpart.)  Bytes the caller must provide for the packed weights arena (persistent layer state:
 * packed codes, params, channel cache, 8-bit pool, switch tables) and for the workspace
 * (scratch of pack and forward; may be shared by several layers whose calls are ordered on
 * one stream).  bits: host int32 [E + E_s], routed experts in {2,3,4,6,8} (the paper's INT2/4/6/8 plus 3),
 * shared experts 8.
 * Host only. */
dynamo_status dynamo_arena_bytes(const dynamo_layer_desc* desc, const int32_t* bits,
                                 size_t* weights_bytes, size_t* workspace_bytes);

/* Offline step: quantize and bit-pack every expert at its assigned bit-width and build the
 * channel cache.  [Section IV-A: expert-level uniform mixed-precision quantization;
 * Section V-B: several low-bit codes packed per 32-bit word; Sections IV-B, V-A: cache of the
 * original channels with (expert, channel) index headers.]
 *   w_gate, w_up : dev bf16 [E+E_s, f, d] row-major;  w_down : dev bf16 [E+E_s, d, f].
 *   bits         : host int32 [E+E_s].
 *   cache_idx    : host int32 [E, P], each row strictly increasing, in [0, d).
 * Per (row, group of G input indices): scale = fp16((max-min)/(2^b-1)) (1.0 if that rounds to 0),
 * zero = fp16(min), code = clamp(rint((w-zero)/scale), 0, 2^b-1), all in IEEE double with ties
 * to even.  For every routed expert with bits < 8 the 8-bit parameters of W_gate/W_up, the 8-bit
 * codes of the P cached channels and their bf16 originals are stored as well.  The significant
 * sets are installed empty.  The arenas must stay valid and unmoved while the context is used.
 * Inputs may be freed once the stream has passed this call. */
dynamo_status dynamo_pack_experts(dynamo_ctx* ctx, const void* w_gate, const void* w_up, const void* w_down,
                                  const int32_t* bits, const int32_t* cache_idx,
                                  void* weights_arena, size_t weights_bytes,
                                  void* workspace, size_t workspace_bytes, void* stream);

/* Runtime channel switch: install the significant-channel set of every routed expert.
 * [Section IV-B: channel replacement from the cache and requantization; Section V-A: lookup by
 * (expert, channel) header.]
 *   sig_idx : host int32 [E, S] (only the first sig_cnt[e] entries of a row are read)
 *   sig_cnt : host int32 [E], each in [0, S].
 * The state afterwards depends only on the sets given (not on history).  Channels must be in the
 * expert's cache (ERR_NOT_CACHED), in range (ERR_INDEX_RANGE), unique (ERR_INDEX_DUP); on any
 * error the previous sets stay installed.  Base codes and params are never touched.  For experts
 * with 8-bit base precision the set is a no-op.  Stream-ordered: a switch enqueued between two
 * forwards takes effect exactly between them. */
dynamo_status dynamo_set_channel_switch(dynamo_ctx* ctx, const int32_t* sig_idx, const int32_t* sig_cnt,
                                        void* stream);

/* A whole switch event (all layers of a stack) in one upload and one launch; all-or-nothing.
 * sig_idx host int32 [n_layers, E, S], sig_cnt host int32 [n_layers, E]; n_layers <= 64; all
 * layers must share shape and workspace. */
dynamo_status dynamo_set_channel_switch_many(dynamo_ctx* const* ctxs, int32_t n_layers,
                                             const int32_t* sig_idx, const int32_t* sig_cnt, void* stream);

/* Select how a switch brings entering channels to 8-bit (DYNAMO_SWITCH_*; default SELECT).
 * Both give bit-identical state. */
dynamo_status dynamo_set_switch_mode(dynamo_ctx* ctx, int32_t mode);

/* Forward of the layer: router top-k -> token permutation -> mixed-precision grouped SwiGLU FFN
 * with the significant-channel correction -> weighted un-permute.  [Section II-A: Top-K expert
 * selection, one-to-many dispatch; Section V-B: packed load, dequantize, tensor-core MMA, fused.]
 *   x             : dev bf16 [T, d], 16-byte aligned (as y must be; misaligned -> ERR_ALIGN)
 *   router_logits : dev fp32 [T, E]   (the router GEMM is outside this path)
 *   y             : dev [T, d], bf16 or fp32 per y_dtype
 * topk = the k largest logits (ties -> lower index), weights = softmax over all E restricted to
 * the chosen k (rescaled to sum 1 if renormalize).  y[t] = sum_j w[t,j] * FFN_{e_j}(x[t]) +
 * sum_shared FFN_s(x[t]), summed in fp32 in that order.  T = 0 is a no-op. */
dynamo_status dynamo_moe_forward(dynamo_ctx* ctx, const void* x, const float* router_logits, int32_t T,
                                 void* y, int32_t y_dtype, const dynamo_debug_out* dbg, void* stream);

/* The same forward with the router's scoring fused in front (Section II-A: the gating network scores every
 * expert for a token, the K best are taken):
 *   logits[t][e] = sum_c x[t][c] * w_router[e][c] + router_bias[e]      (bf16 inputs, fp32 accumulation in a
 *   fixed order: deterministic), then top-k and softmax exactly as above, in the same kernel.
 *   w_router    : dev bf16 [E, d], 16-byte aligned (as x must be)
 *   router_bias : dev fp32 [E] or NULL
 *   logits_out  : dev fp32 [T, E] or NULL: where to store the computed scores (parity tests)
 * Because the scores are rounded in fp32, two experts whose exact scores differ by less than the accumulation
 * error may be ordered differently than by exact arithmetic; given the scores written to logits_out the
 * selection is exactly the rule above.  Errors as dynamo_moe_forward; NULL w_router -> ERR_NULL; misaligned
 * x or w_router -> ERR_ALIGN. */
dynamo_status dynamo_moe_forward_router(dynamo_ctx* ctx, const void* x, const void* w_router,
                                        const float* router_bias, int32_t T, void* y, int32_t y_dtype,
                                        float* logits_out, const dynamo_debug_out* dbg, void* stream);

/* Same forward with HOST buffers: copies x and the logits to the device, runs the forward,
 * copies y back and synchronises the stream before returning.  Pinned host memory makes the
 * copies asynchronous with respect to other streams; pageable memory works too. */
dynamo_status dynamo_moe_forward_host(dynamo_ctx* ctx, const void* x_host, const float* logits_host, int32_t T,
                                      void* y_host, int32_t y_dtype, void* stream);

/* (Utility call: the paper has no counterpart.)  Unpack the stored representation back to logical codes, for parity checks.
 *   q : dev uint8 [out, in] logical codes (row-major, out = f for gate/up, d for down)
 *   scale_f16, zero_f16 : dev uint16 [out, in/G] fp16 bit patterns
 * which = DYNAMO_CODES_*; the HI variants exist for gate/up of routed experts with bits < 8
 * (ERR_BITS otherwise). */
dynamo_status dynamo_export_codes(dynamo_ctx* ctx, int32_t expert, int32_t matrix, uint8_t* q,
                                  uint16_t* scale_f16, uint16_t* zero_f16, int32_t which, void* stream);

/* Algorithmic HBM bytes of one expert per forward (the roofline numerator; the paper has no counterpart): packed
 * base codes + base params of the three matrices, plus (bits < 8) the fp16 tiles of its currently SIGNIFICANT
 * channels, 2 * d_ff * |S_e| * 2 bytes.  What the kernels actually read is a little more: they stream the tiles of
 * the whole cache pool (cache_size channels, zero activations for the ones that are not significant), so that a
 * switch never moves a tile; the difference counts against the achieved fraction as traffic beyond the algorithmic
 * bytes.  Host only (uses the sets last installed). */
dynamo_status dynamo_expert_stream_bytes(dynamo_ctx* ctx, int32_t expert, size_t* bytes);

/* Synchronises the stream, reads the device status word and clears it.  (Utility call: the paper has no
 * counterpart.)  DYNAMO_ERR_TIMEOUT: a bounded device-side wait expired; the kernels of that forward and of every
 * later one started nothing, outputs are undefined until the status is cleared by this call.  DYNAMO_ERR_RANGE: an
 * activation was clamped (see Conventions); outputs are defined.  TIMEOUT wins when both are set.  Else DYNAMO_OK. */
dynamo_status dynamo_poll_status(dynamo_ctx* ctx, void* stream);

/* Debug calls.  (The paper has no counterpart.)
 * dynamo_debug_expire_wait: launches one warp that waits, through the same bounded wait the FFN kernels use but with
 *   limit_ns (1e3 .. 1e8) as its limit, on a barrier that nobody arrives at.  The wait gives up, sets the TIMEOUT
 *   status bit and the kernel returns: nothing faults or hangs.  Exercises the failure path end to end
 *   (dynamo_poll_status reports ERR_TIMEOUT, forwards in between start nothing).
 * dynamo_debug_check_guards: every region of the weights arena and of the workspace is followed by a 256-byte guard
 *   block written at pack time; synchronises the stream and returns in *n_bad_bytes how many guard bytes have changed
 *   since (0 unless a kernel stored outside its region). */
dynamo_status dynamo_debug_expire_wait(dynamo_ctx* ctx, int64_t limit_ns, void* stream);
dynamo_status dynamo_debug_check_guards(dynamo_ctx* ctx, int64_t* n_bad_bytes, void* stream);

/* Operand precision of the tensor-core products (Section V-B dequantizes to FP16; a bf16 pipeline is the other
 * common choice).  Integer codes up to 255 and bf16 inputs are exact in fp16 and in bf16, and every product is exact
 * in the fp32 accumulator, so the two formats differ in ONE place: the hidden activations h = silu(g) * u, which
 * are the second projection's operand.  DYNAMO_OPERAND_FP16 (default) rounds h to fp16 (11 significant bits),
 * DYNAMO_OPERAND_BF16 rounds it to bf16 (8 significant bits; every bf16 value inside the operand range is an fp16
 * value, so the same instruction then computes what bf16 operands give).  Host-side setting, takes effect with the
 * next forward; costs one conversion per hidden value.  Errors: NULL ctx -> ERR_NULL; another value -> ERR_ARG. */
enum { DYNAMO_OPERAND_FP16 = 0, DYNAMO_OPERAND_BF16 = 1 };
dynamo_status dynamo_set_operand_dtype(dynamo_ctx* ctx, int32_t operand_dtype);

/* Path selection: experts that receive more than `rows` tokens in a forward run on the tcgen05
 * (tensor-memory) kernel, the others on the streaming kernel.  Default 32 (also the maximum);
 * 0 switches the tcgen05 path off.  Both paths implement the same arithmetic definition. */
dynamo_status dynamo_set_tc_min_rows(dynamo_ctx* ctx, int32_t rows);

/* Precision the significant channels are served at (Section IV-B: once the original channels are back in place
 * they are requantized to the precision the new data calls for, which may be higher or lower than before).
 *   hi_bits : host int32 [E], each in {2, 3, 4, 6, 8}; 8 for every expert after dynamo_pack_experts.
 * For every routed expert with base bits < 8 whose value changes, one kernel recomputes from the stored group
 * extrema the parameters of the expert's uniform hi_bits[e]-bit quantization of W_gate and W_up (same groups, same
 * quantizer as pack), and from the bf16 channel cache the codes and forward-ready values of all cached channels.
 * A significant channel c then takes the value it has in that quantization; the sets themselves are unchanged.
 * Entries of 8-bit experts are checked but ignored.  Stream-ordered.
 * Errors: NULL -> ERR_NULL; before pack -> ERR_STATE; a value outside the list -> ERR_BITS (nothing changes). */
dynamo_status dynamo_set_channel_precision(dynamo_ctx* ctx, const int32_t* hi_bits, void* stream);

/* Runtime selection of the significant channels on the device (Sections IV-B, V-A: the channels whose dynamics
 * are most prominent under the current data are the ones to switch; only cached channels can be raised).
 *
 * dynamo_set_stats_collection(on): while on, every forward also accumulates, per routed expert e and cached
 *   channel c, A[e][c] += sum over the tokens routed to e in that forward of |x[t][c]| -- in fp32, tokens in
 *   ascending order inside a forward and ONE addition of the forward's sum to the running total, so two runs give
 *   the same bits (the statistics decide an integer selection); against exact sums they carry the fp32
 *   accumulation error n * 2^-24 * A.  One extra kernel per forward.  The paper defines the significance of a
 *   channel only loosely (Section III-A, and Section IV-A's definition of expert significance built on it); the
 *   activation mass of the input channel is the reading taken here.
 * dynamo_get_channel_stats: copies A to stats_out, DEVICE fp32 [E, P] (column j = cached channel cache_idx[e][j]).
 * dynamo_select_significant: per expert with base bits < 8 the n_select (<= max_sig, <= P) cached channels with
 *   the largest A, ties -> lower channel index, become the significant set (slot order = rank order); 8-bit
 *   experts get the empty set.  The tables are rewritten by a device kernel exactly as dynamo_set_channel_switch
 *   would write them, in stream order.  With sig_idx_out and sig_cnt_out both NULL the call does not wait: the
 *   chosen sets travel to a pinned host buffer behind the kernel and the library reads them when the host next
 *   needs them (dynamo_sync_sets, dynamo_expert_stream_bytes, a later switch).  With an output pointer given
 *   (sig_idx_out host [E, max_sig] padded with -1, sig_cnt_out host [E]) the call waits for that copy and fills
 *   them, as dynamo_sync_sets would.  reset != 0 zeroes A.  The first call allocates the pinned buffer and an event.
 * dynamo_sync_sets: waits for the sets of the last dynamo_select_significant (if still on their way) and returns
 *   the sets now installed, whoever installed them; either pointer may be NULL.
 * Errors: NULL ctx -> ERR_NULL; before pack -> ERR_STATE; n_select out of range or a pool too large to rank in
 * shared memory (P > 12288) -> ERR_SHAPE. */
dynamo_status dynamo_set_stats_collection(dynamo_ctx* ctx, int32_t on);
dynamo_status dynamo_get_channel_stats(dynamo_ctx* ctx, float* stats_out, void* stream);
dynamo_status dynamo_select_significant(dynamo_ctx* ctx, int32_t n_select, int32_t reset, int32_t* sig_idx_out,
                                        int32_t* sig_cnt_out, void* stream);
dynamo_status dynamo_sync_sets(dynamo_ctx* ctx, int32_t* sig_idx_out, int32_t* sig_cnt_out);

/* Significant channels on the d_ff side (Section IV-B applied to the second projection: the input channels of
 * W_down are the hidden units).  Optional; a layer that never calls these pays nothing.
 * A significant hidden unit c of routed expert e (base bits < 8) takes column c of the expert's uniform 8-bit
 * quantization of W_down (same groups of G hidden units, same quantizer as dynamo_pack_experts).  The forward
 * realises it as the base down GEMM plus, between that GEMM and the combine, one kernel that adds
 * h[row][c] * (W8[n][c] - Wbase[n][c]) over the significant c, the difference kept as fp16 per (cached channel, n).
 *
 * dynamo_down_cache_bytes: size of the caller-owned arena (256-byte aligned device memory that must outlive the
 *   context's use of it) for cache_size_down cached hidden units per expert and sets of up to max_sig_down.
 * dynamo_pack_down_cache: after dynamo_pack_experts (a new dynamo_pack_experts drops the cache).
 *   w_down         : device bf16 [E + E_s, d_model, d_ff], the originals given to dynamo_pack_experts
 *   cache_idx_down : host int32 [E, cache_size_down], strictly increasing per expert, each in [0, d_ff)
 *   Builds the 8-bit parameters and the extrema of every (row, group) of W_down and, per cached hidden unit, its
 *   8-bit codes, bf16 originals (the channel cache) and differences.  All sets start empty.  Synchronises the stream.
 * dynamo_set_channel_switch_down: installs the sets (the state depends only on the last call).
 *   sig_idx : host int32 [E, max_sig_down], sig_cnt : host int32 [E], 0 <= cnt <= max_sig_down
 *   8-bit experts are validated but keep the empty set.  Stream-ordered like dynamo_set_channel_switch: a switch
 *   enqueued between two forwards takes effect exactly between them (the tables travel by three small copies from
 *   pageable host memory, which the CUDA runtime stages before the call returns).
 *   In switch mode DYNAMO_SWITCH_REQUANT one more kernel re-derives codes and differences of the new sets'
 *   channels from the bf16 channel cache at the expert's target precision (channel replacement followed by
 *   requantization, Section IV-B); the resulting state equals the one DYNAMO_SWITCH_SELECT reaches, bit for bit.
 * dynamo_set_channel_precision_down: precision the significant hidden units are served at (Section IV-B: requantized
 *   to the precision the new data calls for, higher or lower than before); the d_ff-side twin of
 *   dynamo_set_channel_precision, which does not reach this side.
 *   hi_bits : host int32 [E], each in {2, 3, 4, 6, 8}; 8 for every expert after dynamo_pack_down_cache.
 *   For every routed expert with base bits < 8 whose value changes, one kernel recomputes from the stored group
 *   extrema the parameters of the expert's uniform hi_bits[e]-bit quantization of W_down and, from the bf16 channel
 *   cache, the code and the difference to the base value of every cached hidden unit.  A target equal to the base
 *   bit-width makes every difference zero; going back to 8 restores the packed state bit for bit.  Stream-ordered.
 *   Errors: a value outside {2, 3, 4, 6, 8} -> ERR_BITS (nothing changes).
 * dynamo_export_codes with DYNAMO_MAT_DOWN and DYNAMO_CODES_HI_POOL / HI_ACTIVE returns the codes of the cached /
 * significant hidden units at the current target precision (0 elsewhere) and that precision's parameters, shaped
 * like the base export.
 * Errors: NULL -> ERR_NULL; before dynamo_pack_experts (or, for the switch and the export, before
 * dynamo_pack_down_cache) -> ERR_STATE; cache_size_down outside [1, min(d_ff, 65535)], max_sig_down outside
 * [0, min(256, cache_size_down)] -> ERR_SHAPE; arena misaligned -> ERR_ALIGN, too small -> ERR_ARENA_TOO_SMALL; an
 * index outside [0, d_ff) or a count outside its range -> ERR_INDEX_RANGE; a repeated or unsorted index ->
 * ERR_INDEX_DUP; a significant unit that is not cached -> ERR_NOT_CACHED.  On an error the previous state stays. */
dynamo_status dynamo_down_cache_bytes(const dynamo_layer_desc* desc, const int32_t* bits, int32_t cache_size_down,
                                      int32_t max_sig_down, size_t* bytes);
dynamo_status dynamo_pack_down_cache(dynamo_ctx* ctx, const void* w_down, const int32_t* cache_idx_down,
                                     int32_t cache_size_down, int32_t max_sig_down, void* down_arena, size_t down_bytes,
                                     void* stream);
dynamo_status dynamo_set_channel_precision_down(dynamo_ctx* ctx, const int32_t* hi_bits, void* stream);
dynamo_status dynamo_set_channel_switch_down(dynamo_ctx* ctx, const int32_t* sig_idx, const int32_t* sig_cnt,
                                             void* stream);

/* Offline bit-width assignment (Section IV-A, Algorithm 1 and the two paragraphs around it): fuzzy c-means over the
 * experts' significance, clusters mapped to precisions by significance, experts in the overlap of two clusters sent
 * to the lower precision.  HOST code in double precision: every pointer is a host pointer, there is no context, no
 * device work and no stream.  The result can be handed to dynamo_pack_experts (bits) or, after the significance was
 * measured again on new data, to dynamo_set_channel_precision (Section IV-B: the difference between the two
 * clusterings decides the precision the cached channels are requantized to).
 *   x           : [n, dim] significance of each expert (the paper's x_i; dim = 1 there)
 *   c           : number of clusters (the paper: 4), 1 <= c <= min(n, 16)
 *   m, eps      : fuzzifier (> 1) and tolerance (>= 0) of Algorithm 1; the loop ends when the Frobenius norm of
 *                 U_new - U_old is below eps, or after max_iter (>= 1) iterations
 *   u0          : [n, c] initial memberships, every entry in [0, 1], every row summing to 1 (1e-9), or NULL
 *   token_share : [n] each expert's share of the routed tokens, used when u0 is NULL: the initial memberships are
 *                 those of the share against c anchors spread evenly from the smallest to the largest share
 *                 (all equal, or c = 1: 1/c everywhere)
 *   levels      : [c] precision of the most ... least significant cluster, each in {2, 3, 4, 6, 8}
 *   overlap     : >= 0; an expert whose two largest memberships differ by less than this takes the lower of the two
 *                 clusters' precisions (0: plain arg-max; exact ties always resolve to the lower precision)
 * Each iteration: v_k = sum_i u_ik^m x_i / sum_i u_ik^m, then u_ik = 1 / sum_j (|x_i - v_k| / |x_i - v_j|)^(2/(m-1));
 * a point lying on one or more centers shares its membership equally among them.  Clusters are ranked by the mean
 * coordinate of their center (ties: larger membership mass, then lower index).
 * Outputs: bits_out [n]; optional (NULL to skip) cluster_out [n], v_out [c, dim], u_out [n, c], iters_out [1].
 * Errors (outputs untouched): NULL x / levels / bits_out, or u0 and token_share both NULL -> ERR_NULL; n, dim, c or
 * max_iter out of range -> ERR_SHAPE; a level outside the list -> ERR_BITS; m <= 1, eps < 0, overlap < 0, a
 * non-finite value, u0 not row-stochastic, or a cluster left without any membership -> ERR_ARG. */
dynamo_status dynamo_assign_bits(const double* x, int32_t n, int32_t dim, int32_t c, double m, double eps,
                                 int32_t max_iter, const double* u0, const double* token_share,
                                 const int32_t* levels, double overlap, int32_t* bits_out, int32_t* cluster_out,
                                 double* v_out, double* u_out, int32_t* iters_out);

/* Measurement hook: three cudaEvent_t handles (any may be NULL) that every following forward records on
 * its stream before the gate/up FFN launch, after it, and after the down FFN launch, so that a
 * harness can time the dominant kernels in place.  Pass NULLs to switch it off. */
dynamo_status dynamo_set_profile_events(dynamo_ctx* ctx, void* before_gateup, void* after_gateup, void* after_down);

/* Number of kernels the library launched through this context since creation (host counter). */
int64_t dynamo_kernel_launches(const dynamo_ctx* ctx);

const char* dynamo_status_str(dynamo_status s);

/* Routing + permutation for callers that cannot allocate device memory.  (The paper has no
 * counterpart; the step itself is the Top-K selection and one-to-many dispatch of Section II-A.)
 * Some users of this library are not allowed to call cudaMalloc: code that runs while a CUDA graph
 * is being captured, plugins that a framework hands a fixed set of buffers, real-time loops that
 * must stay off the allocator.  dynamo_moe_forward takes its scratch from a workspace the caller
 * allocated; this call needs none: the scan kernel's scratch lives in a fixed array inside the
 * library (about 400 KiB of device memory per GPU that loads the library, held until exit).
 *   router_logits : dev fp32 [T, n_experts]                       (input)
 *   topk_idx      : dev int32 [T, top_k]   topk_w : dev fp32 [T, top_k]
 *   expert_offsets: dev int32 [n_experts + 1]   perm : dev int32 [T * top_k]   (outputs, caller-owned)
 * Same results as the routing outputs of dynamo_moe_forward.  Limits: T * top_k <=
 * DYNAMO_NOALLOC_MAX_PAIRS (ERR_TOKENS beyond), n_experts <= 256, top_k <= 8 (ERR_SHAPE).
 * Calls neither cudaMalloc nor cudaFree nor any allocating routine.  The first call on a device
 * looks up the array's device address (with that device current); make that first call before
 * starting any stream capture.  All calls share the one array, which keeps the previous call's
 * contents (nothing needs clearing: every word read is written first); two calls that overlap on
 * the GPU - different streams, or different threads - race on it, so order them on one stream.
 * T = 0 is a no-op.  Asynchronous and stream-ordered like the other calls. */
#define DYNAMO_NOALLOC_MAX_PAIRS 32768
dynamo_status dynamo_route_permute_static(const float* router_logits, int32_t T, int32_t n_experts, int32_t top_k,
                                          int32_t renormalize, int32_t* topk_idx, float* topk_w,
                                          int32_t* expert_offsets, int32_t* perm, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DYNAMO_H_ */
