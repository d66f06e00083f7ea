// Shared device-side declarations of the DynaMo B200 library: arena descriptors, constants,
// small PTX wrappers (mbarrier, bulk async copy, bounded waits).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dyn {

constexpr int RB = 256;          // weight rows per packed block
constexpr int KC = 128;          // input indices (k) per packed block
constexpr int ATOM_ROWS = 16;    // rows of one MMA fragment tile; a block has 16 atoms
constexpr int XROW = 288;        // bytes per (token row, k-chunk) in activation buffers:
                                 // 128 fp16 + two fp32 sums (k 0..63, 64..127) + pad; 288/4 = 72 = 8 (mod 32) banks
constexpr int XROW_SUM_OFF = 256;
constexpr int POOL_TILE_BYTES = 512;   // one cached channel's 8-bit-valued fp16 column for the 256 rows of a block
constexpr int MAX_EXPERTS = 264;
constexpr int HI_BITS = 8;

// Device status word (bit flags, sticky until dynamo_poll_status clears them).  TIMEOUT: a bounded wait expired,
// later kernels of the stream start nothing.  RANGE: an activation was clamped to the fp16 operand range (the
// forward still completes, with the clamped value).
enum : int { STATUS_OK = 0, STATUS_TIMEOUT = 1, STATUS_RANGE = 2 };

struct ExpertDev {
    const uint8_t* w13;        // packed blocks of the fused gate/up matrix: [n_rb13][n_kc13][blk_bytes]
    const uint8_t* w2;         // packed blocks of the down matrix:          [n_rb2][n_kc2][blk_bytes]
    __half* pool_hi;           // [n_rb13][P + 1][256] fp16, value s8*q8+m8 of cached channel p (tile P = zeros)
    uint32_t* s8m8[2];         // gate, up: [f][d/G] half2 {scale, zero} of the high-precision (hi_bits) quantization
    uint32_t* gminmax[2];      // gate, up: [f][d/G] bf16 pair {min, max} of every group of the original weights
    uint8_t* pool_q8[2];       // gate, up: [P][f] 8-bit codes of the cached channels
    __nv_bfloat16* cache_w[2]; // gate, up: [P][f] bf16 originals of the cached channels (the channel cache)
    int32_t bits;
    int32_t blk_bytes;         // bytes of one packed block (codes + params)
    int32_t switchable;        // routed expert with bits < 8
    int32_t hi_bits;           // precision the significant channels are served at (8 after pack; retargetable)
};

struct LayerDev {
    int32_t d, f, E, Es, k, G, S, S_pad, P, renorm;
    int32_t P_pad;        // P rounded up to a multiple of 32 (tiles beyond P are zero)
    int32_t n_rb13, n_kc13, n_rb2, n_kc2;
    int32_t* cache_idx;   // [E][P] sorted channel indices (cache headers)
    int32_t* sig_chan;    // [E][S_pad] channel of each active slot, -1 = empty
    int32_t* sig_pool;    // [E][S_pad] pool position of each active slot, P = zero tile
    int32_t* sig_cnt;     // [E]
    uint32_t* sigmask;    // [E][d/32] bit c set <=> channel c significant
    int32_t order[MAX_EXPERTS];  // expert ids sorted by descending bits (heaviest work first)
    ExpertDev ex[MAX_EXPERTS];
};

// Significant set on the d_ff side (Section IV-B applied to the input channels of W_down, the hidden units), kept
// in its own caller-owned arena so that layers that do not use it pay nothing.
struct DownExpertDev {
    uint32_t* s8m8;          // [d][f/G] half2 {scale, zero} of W_down's quantization at the target precision (8 after pack)
    uint32_t* gminmax;       // [d][f/G] two bf16 {min, max} of every group: what another target precision is derived from
    uint8_t* q8;             // [P2][d] codes of the cached channels at the target precision
    __half* delta;           // [P2][d] fp16(target value - base value): what a significant channel adds to the base GEMM
    __nv_bfloat16* cache_w;  // [P2][d] bf16 originals of the cached channels (the channel cache)
};
struct DownDev {
    int32_t P2, S2;
    int32_t* cache_idx;  // [E][P2] sorted hidden-unit indices (cache headers)
    int32_t* sig_chan;   // [E][S2] hidden unit of slot i (-1 = empty)
    int32_t* sig_pool;   // [E][S2] pool position of slot i
    int32_t* sig_cnt;    // [E]
    DownExpertDev ex[MAX_EXPERTS];
};

// Workspace pointers of one forward (passed to kernels by value).
struct WsDev {
    int32_t* counts;      // [E_tot]
    int32_t* offsets;     // [E_tot + 1]
    int32_t* topk_idx;    // [T, k]
    float* topk_w;        // [T, k]
    int32_t* perm;        // [T*k]
    int32_t* pos;         // [T, k+Es]  sorted row of pair (t, j)
    int32_t* row_token;   // [R]
    int32_t* row_expert;  // [R]
    uint8_t* xperm;       // [R + pad][d/128][XROW]
    __half* xsig;         // [R + pad][S_pad]
    uint8_t* hbuf;        // [R + pad][f/128][XROW]
    float* ypart;         // [ksplit][Rpad][d] fp32 rows of the down GEMM, one copy per K split
    int32_t* status;      // device status word
    int32_t T, R, ksplit;
    // Physical rows: every expert's segment starts at a multiple of 8 rows (off_pad), so that the
    // tensor-core path can address activations as 8-row groups.  All row-indexed buffers above use
    // physical rows; Rpad is the host-side bound R + 8 * (E + Es).
    int32_t* off_pad;     // [E_tot + 1]
    int32_t Rpad;
    int32_t Rcap;         // rows allocated in the activation buffers (their chunk pitch)
    int32_t tc_min;       // experts with more rows than this take the tcgen05 path (INT_MAX: none)
    int32_t h_bf16;       // 1: hidden activations are rounded to bf16 before they become the down GEMM's operand
};

// Activation layouts.  Both give a row group of 8 rows the same footprint (8 * XROW bytes per 128-k
// chunk), so the two FFN paths can share one buffer:
//   streaming path : row r, chunk c at (r * n_kc + c) * XROW: 128 fp16, then two fp32 sums.
//   tcgen05 path   : row group rg, chunk c at (rg * n_kc + c) * 8 * XROW: the canonical K-major
//                    no-swizzle MMA operand tile [k-octet 16][row 8][k 8] fp16 (2048 B).
constexpr int TC_TILE_BYTES = 2048;
constexpr int TC_RG_STRIDE = 8 * XROW;
constexpr int TC_MIN_ROWS = 32;

// Activation buffers are CHUNK-MAJOR: the 128-k chunk kc of row r sits at (kc * Rcap + r) * XROW, so the
// slice "rows r0 .. r0+n of chunk kc" that one pipeline stage needs is ONE contiguous bulk copy (many small
// copies cost the copy engine about as much each as a large one).  Rcap = allocated rows.
__host__ __device__ __forceinline__ size_t act_off(int kc, int row, int Rcap) {
    return ((size_t)kc * Rcap + row) * XROW;
}
// Gathered activations of the cached ("pool") channels, 32 columns per group pq: (pq * Rcap + r) * 64 bytes.
constexpr int POOL_GROUP = 32;               // cached channels per significant-channel pipeline stage
constexpr int XPOOL_ROW = POOL_GROUP * 2;    // bytes per (row, group)
__host__ __device__ __forceinline__ size_t xpool_off(int pq, int row, int Rcap) {
    return ((size_t)pq * Rcap + row) * XPOOL_ROW;
}
// 8-bit-valued fp16 tiles of the cached channels: [row block][pool position][256 rows], 528-byte pitch
// (the pad keeps ldmatrix rows conflict-free after a contiguous copy); P_pad = P rounded up to 32.
constexpr int POOL_TILE_PITCH = 528;
__host__ __device__ __forceinline__ size_t pool_tile_off(int rb, int p, int P_pad) {
    return ((size_t)rb * P_pad + p) * POOL_TILE_PITCH;
}

// Layers of one switch event (kernel parameter).
struct SwitchLayers {
    const LayerDev* layer[64];
};

// The MMA operands are fp16 and carry a power-of-two pre-scale of at most 2^4, so an activation (an input x or a
// hidden value h) must satisfy |v| * 16 <= 65504.  Magnitudes above ACT_LIMIT = 4080 (the largest value below
// 65504 / 16 that both bf16 and fp16 hold exactly; infinities included) are clamped to +-ACT_LIMIT and reported
// through STATUS_RANGE; NaN passes through.
constexpr float ACT_LIMIT = 4080.f;
__device__ __forceinline__ float clamp_act(float v, bool& hit) {
    if (fabsf(v) > ACT_LIMIT) {
        hit = true;
        v = copysignf(ACT_LIMIT, v);
    }
    return v;
}

// Operand precision of the hidden activations.  The integer codes (at most 255) and the bf16 inputs are exact in
// fp16 and in bf16 alike and every product is exact in the fp32 accumulator, so the hidden value h is the one
// operand on which a bf16 tensor-core path and an fp16 one differ: rounding h to bf16 (an exact fp16 value inside
// the clamp range) gives the arithmetic of bf16 operands on the fp16 instruction.
__device__ __forceinline__ float round_operand(float h, int to_bf16) {
    return to_bf16 ? __bfloat162float(__float2bfloat16_rn(h)) : h;
}

// ---- PTX helpers -----------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Cluster forms (thread-block clusters of two CTAs driving one tensor-core pair).
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
}
// Arrive on the barrier at the same shared-memory offset in CTA `cta` of the cluster.  Default semantics on
// purpose: what these arrivals hand over is the COMPLETION of asynchronous work (tensor-memory stores and loads
// waited for with tcgen05.wait, bulk copies observed on their own barrier), not generic-proxy data, so no
// cluster-scope fence is needed; an explicit .release.cluster here (and .acquire.cluster on the waiting side) cost
// the pair kernel a fifth of its time.
__device__ __forceinline__ void mbar_arrive_remote(uint64_t* bar, uint32_t cta) {
    asm volatile(
        "{\n\t.reg .b32 ra;\n\tmapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.shared::cluster.b64 _, [ra];\n\t}" ::"r"(smem_u32(bar)),
        "r"(cta)
        : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// The same poll with a suspend-time hint (ns): the hardware may park the thread up to that long before it reports
// a phase that has not completed, so a waiting warp issues fewer polls.
__device__ __forceinline__ bool mbar_try_wait_hint(uint64_t* bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait: spins on the barrier phase for at most ~1 s.  On expiry (or when another thread of
// the CTA already gave up) it records STATUS_TIMEOUT, raises the CTA-wide poison flag and returns
// false; callers then leave their loops.
constexpr unsigned long long WAIT_LIMIT_NS = 1000ull * 1000ull * 1000ull;
// `where` / `aux` identify the wait: the first waiter of a launch to give up leaves (where, block, thread, aux)
// in words 8..11 of the status block for the host to read.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* poison,
                                                  int32_t* status, unsigned long long limit_ns = WAIT_LIMIT_NS,
                                                  int where = 0, int aux = 0) {
    if (mbar_try_wait(bar, parity)) return true;
    // The clock is read only every 1024 failed polls (a poll itself suspends for a while in hardware):
    // reading %globaltimer on every wait that does not pass at once costs far more than the wait.
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    while (true) {
        if (mbar_try_wait_hint(bar, parity, 20000u)) return true;
        if ((++spins & 0x3ff) == 0) {
            if (*poison) return false;
            const unsigned long long now = globaltimer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > limit_ns) {
                *poison = 1;
                if (atomicCAS(status + 8, 0, where | 0x1000) == 0) {
                    status[9] = (int)blockIdx.x;
                    status[10] = (int)threadIdx.x;
                    status[11] = aux;
                }
                atomicOr(status, STATUS_TIMEOUT);
                return false;
            }
        }
    }
}

// The same wait for barriers that threads of the peer CTA arrive on (default acquire: see mbar_arrive_remote).
__device__ __forceinline__ bool mbar_wait_bounded_cluster(uint64_t* bar, uint32_t parity, volatile int* poison,
                                                          int32_t* status) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    while (true) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((++spins & 0x3ff) == 0) {
            if (*poison) return false;
            const unsigned long long now = globaltimer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > WAIT_LIMIT_NS) {
                *poison = 1;
                atomicOr(status, STATUS_TIMEOUT);
                return false;
            }
        }
    }
}

// 1-D bulk async copy global -> shared, completion counted on an mbarrier (bytes % 16 == 0,
// both addresses 16-byte aligned).
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(smem_dst)),
        "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// m16n8k16 fp16 x fp16 -> fp32
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// ---- programmatic dependent launch -----------------------------------------------------------
// Every kernel of a forward is launched with the programmatic-stream-serialization attribute and
// starts with pdl_prologue(): it lets the next kernel's CTAs be scheduled early (they park in their
// own pdl_prologue) and then waits until the preceding kernel has completed and flushed its
// memory, so launch latency overlaps the previous kernel's tail without changing the data flow.
__device__ __forceinline__ void pdl_prologue() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// The same, as clusters of `cluster` CTAs along x (grid.x must be a multiple of it).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, unsigned cluster,
                                      cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = cluster;
    at[1].val.clusterDim.y = 1;
    at[1].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// ---- packed-block geometry ---------------------------------------------------------------

__host__ __device__ __forceinline__ int atom_bytes(int bits) { return 256 * bits; }  // 16 rows x 128 k
__host__ __device__ __forceinline__ int block_code_bytes(int bits) { return 4096 * bits; }
__host__ __device__ __forceinline__ int block_bytes(int bits, int G) { return 4096 * bits + RB * (KC / G) * 4; }

// Row of the fused gate/up matrix: block rb, atom a, row ra (0..15): rows 0..7 of an atom are gate
// rows, rows 8..15 the up rows of the same eight hidden indices h = 128*rb + 8*a + (ra & 7).
__host__ __device__ __forceinline__ int w13_hidden_index(int rb, int r) {
    return 128 * rb + 8 * (r >> 4) + (r & 7);
}
__host__ __device__ __forceinline__ int w13_row_in_block(int h, int is_up) {
    return 16 * ((h & 127) >> 3) + (h & 7) + (is_up ? 8 : 0);
}

}  // namespace dyn
