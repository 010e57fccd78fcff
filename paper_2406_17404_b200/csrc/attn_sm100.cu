// Tree-masked attention for sm_100a (bf16, head_dim 128, up to 128 tree rows per sequence).
//
// Work is cut into units of one 128-key tile of one (sequence, head); the units, laid out sequence-
// major, are dealt in equal contiguous ranges to a persistent grid of one CTA per SM, so a long prefix
// is split over several CTAs (split-KV) and short sequences are packed several per CTA.  Inside a CTA:
//   * one thread streams Q (per segment) and the K/V tiles with TMA into 128-byte-swizzled shared memory;
//   * one thread issues tcgen05.mma: S = Q.K^T into TMEM (two S buffers), then O += P.V with P read from
//     TMEM as well (two P buffers) and the accumulator resident in TMEM for the whole segment;
//   * eight (or sixteen) warps do the softmax: a thread owns half (a quarter) of one query row (TMEM lane = row, 64 of the 128
//     columns); they read S once into registers, apply the ancestor bitmask on tiles that reach the tree
//     rows, keep an online softmax whose running maximum is only raised when a tile exceeds it by more
//     than 2^8 (then O is rescaled in TMEM), and store P as bf16 pairs back into TMEM, where the second
//     MMA reads it as its A operand: the softmax of a tile never waits for the previous tile's P.V.
// A segment that covers all tiles of its (sequence, head) writes the normalised bf16 output itself;
// otherwise it leaves (max, sum, O) in the workspace and a second kernel merges the pieces in a fixed
// order.  Every wait on an mbarrier is bounded; on expiry the CTA records TRJ_ETIMEOUT and leaves.
#include <cuda.h>
#include <cstdlib>
#include <mutex>
#include "trj_internal.h"
#include "sm100_common.cuh"
#include "timeline.cuh"

namespace trj {
namespace {

constexpr int AT_ROWS = 128;                 // query rows per CTA = UMMA M = TMEM lanes
constexpr int AT_KEYS = 128;                 // keys per tile
constexpr int AT_D = 128;                    // head_dim
// The softmax is done by 4 * SPLIT warps: SPLIT threads share a query row, each taking a column group of a tile
// (template parameter of the kernel: 2 for one sequence with full row groups, 4 for batches of small trees, where
// half of the row groups are empty and more threads per row pay off).
__host__ __device__ constexpr int at_threads(int split) { return 32 * 4 * split + 64; }   // softmax warps + TMA warp + MMA warp
constexpr uint32_t AT_SUB = 128 * 128;       // one [128 x 64 bf16] swizzled sub-tile: 16 KB
constexpr uint32_t AT_TILE = 2 * AT_SUB;     // Q, P, a K tile or a V tile: 32 KB
constexpr int AT_RING = 5;                   // K/V ring slots; load n = 2g + (0: K, 1: V) of tile g goes to slot n % 5
constexpr uint32_t AT_SMEM = (1 + AT_RING) * AT_TILE + 1024;
constexpr float AT_RESCALE_GAP = 8.f;        // raise the running max only when exceeded by 2^8
constexpr int AT_PIECE_STRIDE = AT_D + 4;      // floats per row of a piece in shared memory (16-byte stores without bank conflicts)
constexpr size_t AT_SLOT_FLOATS = (size_t)AT_D * AT_ROWS + 2 * AT_ROWS;   // O^T [d][row], m[row], l[row]

// barrier indices
enum { B_KV_FULL = 0, B_KV_EMPTY = 5, B_Q_FULL = 10, B_Q_EMPTY = 11, B_S_FULL = 12, B_P_READY = 14, B_P_FREE = 16,
       B_O_READY = 18, B_O_FREE = 19, B_COUNT = 20 };

struct AtParams {
    const int32_t* seq_len; const int32_t* row_off; const uint64_t* anc;
    int anc_words, B, H, max_seq;
    int Hkv, group;              // K/V heads and query heads per K/V head (grouped-query attention; group = 1: multi-head)
    __nv_bfloat16* out;          // [rows_total][H][128]
    __nv_bfloat16* out_lo;       // optional: rounding error of `out` as a second bf16 tensor (same shape)
    float* slots;                // partial results, AT_SLOT_FLOATS each
    int* status;
    float scale_log2;            // log2(e) / sqrt(D)
    int cluster;                 // CTAs per thread-block cluster that share one head (1: no clusters)
    int early_ok;                // cache rows below seq_len are older than the chain: they may be fetched before the wait
    int shared_cache;            // every sequence of the batch uses the cache of sequence 0 (pieces of one prompt chunk)
};

using namespace sm100;

// MN-major operand (V: keys are the contraction dim, head_dim is contiguous): 64-element spans of the
// MN dim are 128-byte rows, one per key; 8-key groups 1024 bytes apart (stride offset); the second
// 64-element block of the MN dim lies one sub-tile further (leading offset).
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr) {
    return (uint64_t)((addr & 0x3FFFF) >> 4) | ((uint64_t)(AT_SUB >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Eight MMAs in one go.  A single thread issues them, and its integer work per MMA is what limits the tile loop,
// so the descriptors are not rebuilt: the high words are constants and a step along the contraction dimension
// only adds to the start-address field of the low word (the operands stay inside one 256 KB window).
// S = Q.K^T for one tile: both operands K-major; step kk adds (kk / 4) sub-tiles + (kk % 4) * 32 bytes.
#define TRJ_MMA_SS(step, pred)                                                            \
    "add.u32 al, %1, " #step ";\n\tadd.u32 bl, %2, " #step ";\n\t"                        \
    "mov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"                                  \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, " #pred ";\n\t"
__device__ __forceinline__ void umma8_qk(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc) {
    asm volatile("{\n\t.reg .pred pt, pf;\n\t.reg .b32 al, bl;\n\t.reg .b64 da, db;\n\t"
                 "setp.eq.b32 pt, 0, 0;\n\tsetp.ne.b32 pf, 0, 0;\n\t"
                 TRJ_MMA_SS(0, pf) TRJ_MMA_SS(2, pt) TRJ_MMA_SS(4, pt) TRJ_MMA_SS(6, pt)
                 TRJ_MMA_SS(1024, pt) TRJ_MMA_SS(1026, pt) TRJ_MMA_SS(1028, pt) TRJ_MMA_SS(1030, pt)
                 "}"
                 ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc) : "memory");
}
#undef TRJ_MMA_SS
// O (+)= P.V for one tile: P from tensor memory (16 keys = 8 columns per step), V MN-major (16 keys = 2048 bytes per step).
#define TRJ_MMA_TS(kk, pred)                                                              \
    "add.u32 ta, %1, " #kk "*8;\n\tadd.u32 bl, %2, " #kk "*128;\n\t"                      \
    "mov.b64 db, {bl, %3};\n\t"                                                            \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %4, " #pred ";\n\t"
__device__ __forceinline__ void umma8_pv(uint32_t tmem_d, uint32_t tmem_a, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                         uint32_t accumulate_first) {
    asm volatile("{\n\t.reg .pred pt, pf;\n\t.reg .b32 ta, bl;\n\t.reg .b64 db;\n\t"
                 "setp.eq.b32 pt, 0, 0;\n\tsetp.ne.b32 pf, %5, 0;\n\t"
                 TRJ_MMA_TS(0, pf) TRJ_MMA_TS(1, pt) TRJ_MMA_TS(2, pt) TRJ_MMA_TS(3, pt)
                 TRJ_MMA_TS(4, pt) TRJ_MMA_TS(5, pt) TRJ_MMA_TS(6, pt) TRJ_MMA_TS(7, pt)
                 "}"
                 ::"r"(tmem_d), "r"(tmem_a), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate_first) : "memory");
}
#undef TRJ_MMA_TS
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// Two back-to-back 32-column loads with one wait (64 consecutive columns).
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, float* v) {
    uint32_t r[64];
#define TRJ_LD32(base, off)                                                                                          \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                           \
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "                            \
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"            \
                 : "=r"(r[off + 0]), "=r"(r[off + 1]), "=r"(r[off + 2]), "=r"(r[off + 3]), "=r"(r[off + 4]), "=r"(r[off + 5]),   \
                   "=r"(r[off + 6]), "=r"(r[off + 7]), "=r"(r[off + 8]), "=r"(r[off + 9]), "=r"(r[off + 10]), "=r"(r[off + 11]), \
                   "=r"(r[off + 12]), "=r"(r[off + 13]), "=r"(r[off + 14]), "=r"(r[off + 15]), "=r"(r[off + 16]),               \
                   "=r"(r[off + 17]), "=r"(r[off + 18]), "=r"(r[off + 19]), "=r"(r[off + 20]), "=r"(r[off + 21]),               \
                   "=r"(r[off + 22]), "=r"(r[off + 23]), "=r"(r[off + 24]), "=r"(r[off + 25]), "=r"(r[off + 26]),               \
                   "=r"(r[off + 27]), "=r"(r[off + 28]), "=r"(r[off + 29]), "=r"(r[off + 30]), "=r"(r[off + 31])                \
                 : "r"(base) : "memory")
    TRJ_LD32(taddr, 0);
    TRJ_LD32(taddr + 32, 32);
#undef TRJ_LD32
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
                 "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                 ::"r"(taddr),
                   "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
                   "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
                   "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
                   "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
                   "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
                   "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
                   "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
                   "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
                 : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st32u(uint32_t taddr, const uint32_t* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
                 "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                 ::"r"(taddr),
                   "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                   "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
                   "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
                   "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
                 : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st16u(uint32_t taddr, const uint32_t* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                   "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
                 : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);      // .x (low half) = a
    return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float bf16_round(float a) { return __bfloat162float(__float2bfloat16_rn(a)); }
// Stores 8 consecutive outputs as bf16 (16 bytes) and, when asked, the rounding errors as a second bf16 vector.
__device__ __forceinline__ void store8_split(__nv_bfloat16* hi, __nv_bfloat16* lo, const float* v) {
    *reinterpret_cast<uint4*>(hi) = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
    if (lo) {
        float r[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) r[i] = v[i] - bf16_round(v[i]);
        *reinterpret_cast<uint4*>(lo) = make_uint4(pack_bf16(r[0], r[1]), pack_bf16(r[2], r[3]), pack_bf16(r[4], r[5]), pack_bf16(r[6], r[7]));
    }
}

// Same for 4 outputs (8 bytes each).
__device__ __forceinline__ void store4_split(__nv_bfloat16* hi, __nv_bfloat16* lo, float a, float b, float c, float d) {
    *reinterpret_cast<uint2*>(hi) = make_uint2(pack_bf16(a, b), pack_bf16(c, d));
    if (lo)
        *reinterpret_cast<uint2*>(lo) = make_uint2(pack_bf16(a - bf16_round(a), b - bf16_round(b)),
                                                   pack_bf16(c - bf16_round(c), d - bf16_round(d)));
}
// Distributed shared memory: the address of `local` (a shared::cta address) in CTA `rank` of the cluster, and loads from it.
__device__ __forceinline__ uint32_t cluster_addr(uint32_t local, int rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ float ld_cluster(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float4 ld_cluster4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// 128-bit (lo, hi) shifts by 0..127 bits; the left shift fills the vacated low bits with ones.
__device__ __forceinline__ void shr128(uint64_t& lo, uint64_t& hi, int n) {
    if (n == 0) return;
    if (n < 64) { lo = (lo >> n) | (hi << (64 - n)); hi >>= n; }
    else { lo = hi >> (n - 64); hi = 0; }
}
__device__ __forceinline__ void shl128_fill(uint64_t& lo, uint64_t& hi, int n) {
    if (n == 0) return;
    if (n < 64) { hi = (hi << n) | (lo >> (64 - n)); lo = (lo << n) | ((1ull << n) - 1); }
    else { hi = (n == 64 ? lo : (lo << (n - 64)) | ((1ull << (n - 64)) - 1)); lo = ~0ull; }
}

// Where a unit index falls: sequence, head, tile, and the geometry of that sequence.
struct Where { int b, h, t, tiles, S, rows, bh; };

struct Sched {
    int B, H;
    int tiles[TRJ_MAX_BATCH];           // key tiles of each sequence
    int S[TRJ_MAX_BATCH];               // cached rows of each sequence (a copy of seq_len: no global load on the critical path)
    int row0[TRJ_MAX_BATCH + 1];        // a copy of row_off
    int first[TRJ_MAX_BATCH + 1];       // first unit of each sequence (the launcher checks that the count fits an int)
    int u_begin, u_end;                 // this CTA's units
    __device__ void locate(int u, Where& w) const {
        int b = 0;
        while (b + 1 < B && u >= first[b + 1]) ++b;
        const int r = u - first[b];
        w.b = b; w.tiles = tiles[b];
        w.h = r / w.tiles; w.t = r % w.tiles;
        w.S = S[b]; w.rows = row0[b + 1] - row0[b];
        w.bh = b * H + w.h;
    }
};

__device__ __forceinline__ void build_sched(Sched& s, const AtParams& p) {
    s.B = p.B; s.H = p.H;
    int u = 0;
    s.row0[0] = p.row_off[0];
    for (int b = 0; b < p.B; ++b) {
        s.row0[b + 1] = p.row_off[b + 1];
        // a device-held length that breaks the caller's contract must not turn into a negative or unbounded tile
        // count: it is brought inside the cache (the tensor maps read zeros past the cache's end anyway)
        const int rows_b = min(max(s.row0[b + 1] - s.row0[b], 0), AT_ROWS);
        s.S[b] = min(max(p.seq_len[b], 0), max(p.max_seq - rows_b, 0));
        const int total = s.S[b] + rows_b;
        s.tiles[b] = (total + AT_KEYS - 1) / AT_KEYS;
        s.first[b] = u;
        u += s.tiles[b] * p.H;
    }
    s.first[p.B] = u;
}
// The calling CTA's units.  Without clusters: equal contiguous ranges of all units.  With clusters (one sequence,
// one head per cluster): the head's tiles are shared out among the CTAs of the cluster.
__device__ __forceinline__ void build_range(Sched& s, const AtParams& p) {
    if (p.cluster > 1) {
        const int head = blockIdx.x / p.cluster, rank = blockIdx.x % p.cluster, T = s.tiles[0];
        // shares rounded so that the extra tiles go to the FIRST CTAs: their tiles are cached rows that are already
        // on their way when the previous kernel ends, while the last CTA has the tile with this step's rows, the
        // masks and the padding to deal with
        s.u_begin = head * T + (T * rank + p.cluster - 1) / p.cluster;
        s.u_end = head * T + (T * (rank + 1) + p.cluster - 1) / p.cluster;
    } else {
        const long long U = s.first[p.B];
        s.u_begin = (int)(U * blockIdx.x / gridDim.x);
        s.u_end = (int)(U * (blockIdx.x + 1) / gridDim.x);
    }
}

// PRECISE: the probabilities go to the second product as a bf16 pair hi + lo (lo = the rounding error of hi, kept in
// the tile's own score buffer once the scores are in registers), so the product sees ~16 mantissa bits of P.  A
// single bf16 P costs ~1e-3 of relative error in the output whatever the number of keys (the output of near-uniform
// attention is a mean of n values and the rounding errors of its n weights do not average out any faster than it
// does); inside a deep decoder that error flips the bf16 roundings of the next layers' K/V rows and grows with depth.
template <int AT_SPLIT, bool PRECISE>
__global__ void __launch_bounds__(at_threads(AT_SPLIT), 1) tree_attention_tc_kernel(const __grid_constant__ CUtensorMap map_q,
                                                                          const __grid_constant__ CUtensorMap map_k,
                                                                          const __grid_constant__ CUtensorMap map_v,
                                                                          const AtParams p) {
    constexpr int AT_KPT = 128 / AT_SPLIT;        // keys of a tile, and head_dim columns of O, per thread
    constexpr int AT_SM_WARPS = 4 * AT_SPLIT;     // warp w owns TMEM lanes 32*(w%4).. and column group w/4
    constexpr int AT_SM_THREADS = 32 * AT_SM_WARPS;
    constexpr int AT_W_COPY = AT_SM_WARPS, AT_W_MMA = AT_SM_WARPS + 1;
    constexpr int AT_THREADS = at_threads(AT_SPLIT);
    static_assert(AT_KPT == 32 || AT_KPT == 64, "column groups are read with 32- or 64-column tensor-memory loads");
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[B_COUNT];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ Sched sched;
    __shared__ float pair_max[2][AT_SPLIT][AT_ROWS], pair_sum[2][AT_SPLIT][AT_ROWS];      // [parity][column group][row]
    __shared__ float piece_m[AT_ROWS], piece_l[AT_ROWS];                     // this CTA's piece of a head shared by a cluster

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t q_smem = base, ring_smem = base + AT_TILE;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    pdl_launch_dependents();
    TRJ_TL_DECL;
    if (threadIdx.x == 32) {                                 // have the tensor maps on their way before the first copy needs them
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    }
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int i = 0; i < B_COUNT; ++i)
            mbar_init(bar(i), (i == B_P_READY || i == B_P_READY + 1 || i == B_O_FREE) ? AT_SM_THREADS : 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == AT_W_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Barriers, TMEM and the schedule are set up while the previous kernel may still run: the batch geometry is
    // older than the chain this kernel is launched in.  So are the cache rows below seq_len, which the copy thread
    // starts to fetch before it waits; everything else (q, the tree's own K/V rows) is touched after the wait.
    if (threadIdx.x == 0) { build_sched(sched, p); build_range(sched, p); }
    if (threadIdx.x < AT_ROWS) piece_m[threadIdx.x] = -INFINITY;             // no piece yet
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // Every role works out its first segment before it waits for the previous kernel (one thread's integer
    // divisions and address arithmetic take a microsecond that would otherwise sit on the critical path).
    const uint32_t tmem = tmem_base_slot;
    // TMEM columns: S buffers 0-127 and 128-255, O 256-383, P buffers (bf16 pairs, 64 columns each) 384-447 and 448-511
    const uint32_t tmem_s[2] = {tmem, tmem + 128}, tmem_o = tmem + 256, tmem_p[2] = {tmem + 384, tmem + 448};
    const int u_begin = sched.u_begin, u_end = sched.u_end;
    // With clusters every CTA leaves its piece in its own shared memory, and after a cluster barrier each CTA
    // merges a slice of head_dim from all pieces.
    float* piece_o = reinterpret_cast<float*>(base_ptr + AT_TILE);          // [row][AT_PIECE_STRIDE], over the K/V ring once it is idle

    if (warp == AT_W_COPY) {
        if (lane == 0) {
            // ------------------------------------------------ TMA producer
            int g = 0, e = 0;
            bool ok = true;
            bool waited = false;                             // for the previous kernel (see above)
            const uint64_t kv_policy = l2_evict_first_policy();
            if (!p.early_ok) { pdl_wait(); waited = true; }
            for (int u = u_begin; u < u_end && ok;) {
                Where w; sched.locate(u, w);
                const int t_end = min(w.tiles, w.t + (u_end - u));
                // Q of this segment (after the previous segment's S = Q.K^T products have finished)
                auto load_q = [&]() -> bool {
                    if (!mbar_wait(bar(B_Q_EMPTY), (uint32_t)(e & 1) ^ 1u, &abort_flag, p.status)) return false;
                    mbar_expect_tx(bar(B_Q_FULL), AT_TILE);
                    tma_load_2d(q_smem, &map_q, w.h * AT_D, sched.row0[w.b], bar(B_Q_FULL));
                    tma_load_2d(q_smem + AT_SUB, &map_q, w.h * AT_D + 64, sched.row0[w.b], bar(B_Q_FULL));
                    return true;
                };
                // the first segment's Q is requested by the MMA thread as soon as the previous kernel is done, so
                // that it does not queue behind the cache tiles this thread asks for ahead of the wait
                if (e > 0) { ok = load_q(); if (!ok) break; }
                const int cache_row0 = ((p.shared_cache ? 0 : w.b) * p.Hkv + w.h / p.group) * p.max_seq;
                const int old_tiles = w.S / AT_KEYS;          // tiles that hold cached rows only
                for (int t = w.t; t < t_end && ok; ++t, ++g) {
                    for (int kv = 0; kv < 2 && ok; ++kv) {
                        // rows of this step, or a ring slot that is only freed once Q has arrived: bounded waits
                        // must not start while the previous kernel may still run
                        if (!waited && (t >= old_tiles || 2 * g + kv >= AT_RING)) { pdl_wait(); waited = true; }
                        const int slot = (2 * g + kv) % AT_RING;
                        const uint32_t phase = (uint32_t)((2 * g + kv) / AT_RING) & 1u;
                        ok = mbar_wait(bar(B_KV_EMPTY + slot), phase ^ 1u, &abort_flag, p.status);
                        if (!ok) break;
                        const uint32_t dst = ring_smem + slot * AT_TILE;
                        mbar_expect_tx(bar(B_KV_FULL + slot), AT_TILE);
                        const CUtensorMap* map = kv ? &map_v : &map_k;
                        tma_load_2d_hint(dst, map, 0, cache_row0 + t * AT_KEYS, bar(B_KV_FULL + slot), kv_policy);
                        tma_load_2d_hint(dst + AT_SUB, map, 64, cache_row0 + t * AT_KEYS, bar(B_KV_FULL + slot), kv_policy);
                    }
                }
                if (!waited) { pdl_wait(); waited = true; }  // the next segment's Q comes from the previous kernel
                u += t_end - w.t;
                ++e;
            }
            if (!waited) pdl_wait();
        }
    } else if (warp == AT_W_MMA) {
        if (lane == 0) {
            // ------------------------------------------------ MMA issuer
            // S = Q.K^T: both K-major from shared memory, 128 x 128.  O += P.V: P from TMEM, V MN-major, 128 x 128.
            const uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(AT_KEYS >> 3) << 17) | ((uint32_t)(AT_ROWS >> 4) << 24);
            const uint32_t idesc_pv = idesc_qk | (1u << 16);
            int g = 0, e = 0;
            bool ok = true;
            auto issue_qk = [&](int gg) -> bool {
                const int slot = (2 * gg) % AT_RING;
                if (!mbar_wait(bar(B_KV_FULL + slot), (uint32_t)((2 * gg) / AT_RING) & 1u, &abort_flag, p.status)) return false;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t k_smem = ring_smem + slot * AT_TILE;
                // 8 x 16 elements of head_dim: two sub-tiles of four steps
                const uint64_t q_desc = desc_kmajor_sw128(q_smem), k_desc = desc_kmajor_sw128(k_smem);
                umma8_qk(tmem_s[gg & 1], (uint32_t)q_desc, (uint32_t)k_desc, (uint32_t)(q_desc >> 32), idesc_qk);
                umma_commit(bar(B_S_FULL + (gg & 1)));
                umma_commit(bar(B_KV_EMPTY + slot));
                return true;
            };
            for (int u = u_begin; u < u_end && ok;) {
                Where w; sched.locate(u, w);
                const int n_tiles = min(w.tiles - w.t, u_end - u);
                const int g0 = g, g1 = g + n_tiles;
                if (e == 0) {                                // first segment: Q as soon as the previous kernel is done
                    pdl_wait();
                    mbar_expect_tx(bar(B_Q_FULL), AT_TILE);
                    tma_load_2d(q_smem, &map_q, w.h * AT_D, sched.row0[w.b], bar(B_Q_FULL));
                    tma_load_2d(q_smem + AT_SUB, &map_q, w.h * AT_D + 64, sched.row0[w.b], bar(B_Q_FULL));
                }
                ok = mbar_wait(bar(B_Q_FULL), (uint32_t)(e & 1), &abort_flag, p.status);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                ok = issue_qk(g0);
                for (g = g0; g < g1 && ok; ++g) {
                    if (g + 1 < g1) ok = issue_qk(g + 1);
                    else umma_commit(bar(B_Q_EMPTY));        // every S product of the segment has been issued
                    if (!ok) break;
                    ok = mbar_wait(bar(B_P_READY + (g & 1)), (uint32_t)(g >> 1) & 1u, &abort_flag, p.status);
                    if (ok && g == g0 && e > 0) ok = mbar_wait(bar(B_O_FREE), (uint32_t)((e - 1) & 1), &abort_flag, p.status);
                    const int slot = (2 * g + 1) % AT_RING;
                    if (ok) ok = mbar_wait(bar(B_KV_FULL + slot), (uint32_t)((2 * g + 1) / AT_RING) & 1u, &abort_flag, p.status);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t v_smem = ring_smem + slot * AT_TILE;
                    // 8 x 16 keys; P comes straight from TMEM
                    const uint64_t v_desc = desc_mnmajor(v_smem);
                    umma8_pv(tmem_o, tmem_p[g & 1], (uint32_t)v_desc, (uint32_t)(v_desc >> 32), idesc_pv, g > g0 ? 1u : 0u);
                    if constexpr (PRECISE)                   // the low halves of P sit in the first 64 columns of the tile's S buffer
                        umma8_pv(tmem_o, tmem_s[g & 1], (uint32_t)v_desc, (uint32_t)(v_desc >> 32), idesc_pv, 1u);
                    umma_commit(bar(B_P_FREE + (g & 1)));
                    umma_commit(bar(B_KV_EMPTY + slot));
                }
                if (ok) umma_commit(bar(B_O_READY));
                u += n_tiles;
                ++e;
            }
        }
    } else {
        // ------------------------------------------------ softmax + epilogue
        // Warp w owns rows 32*(w%4) .. +31 (its TMEM lanes) and key / head_dim columns AT_KPT*(w/4) .. +AT_KPT-1, so
        // AT_SPLIT threads share a row and exchange their maxima and sums through shared memory.
        const int rg = warp & 3, part = warp >> 2;
        const int row = rg * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(rg * 32) << 16;
        const uint32_t col0 = (uint32_t)part * AT_KPT;
        const uint32_t pair_bar = 1 + rg;                    // named barrier of the warps of a row group
        int g = 0, e = 0;
        bool ok = true;
        for (int u = u_begin; u < u_end && ok;) {
            Where w; sched.locate(u, w);
            const int n_tiles = min(w.tiles - w.t, u_end - u);
            const int g0 = g, g1 = g + n_tiles;
            const bool live = row < w.rows;
            const bool group_live = rg * 32 < w.rows;        // same for both warps of the pair
            const int grow = sched.row0[w.b] + row;           // global row (valid when live)
            uint64_t m0 = 0, m1 = 0;
            if (live) {
                m0 = p.anc[(size_t)grow * p.anc_words];
                if (p.anc_words > 1) m1 = p.anc[(size_t)grow * p.anc_words + 1];
            }
            const int total = w.S + w.rows;
            float m_ref = -INFINITY, l_sum = 0.f;
            if (e == 0) { pdl_wait(); TRJ_TL_BEGIN(TRJ_TL_ATTENTION); }      // the ancestor masks above are older than the chain
            for (g = g0; g < g1 && ok; ++g) {
                const int key0 = (w.t + (g - g0)) * AT_KEYS;
                const bool edge = key0 + AT_KEYS > w.S;      // the tile reaches tree rows or the end of the keys
                float s[AT_KPT];
                float mt = -INFINITY;
                if (group_live) {
                    ok = __all_sync(0xffffffffu, mbar_wait(bar(B_S_FULL + (g & 1)), (uint32_t)(g >> 1) & 1u, &abort_flag, p.status));
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    if constexpr (AT_KPT == 64) tmem_ld64(tmem_s[g & 1] + lane_addr + col0, s);
                    else tmem_ld32(tmem_s[g & 1] + lane_addr + col0, s);
                    if (edge) {
                        // bit c of (vis0, vis1) = visibility of key key0 + c for this row: tree row tt = key0 + c - S
                        // is visible if tt < 0 (prefix) or if bit tt of the row's ancestor mask is set
                        uint64_t vis0 = m0, vis1 = m1;
                        const int d = key0 - w.S;            // -127 .. 127 on an edge tile
                        if (d >= 0) shr128(vis0, vis1, d); else shl128_fill(vis0, vis1, -d);
                        const uint64_t vis = (col0 < 64 ? vis0 : vis1) >> (col0 & 63u);      // this thread's AT_KPT keys
#pragma unroll
                        for (int i = 0; i < AT_KPT; ++i) if (!((vis >> i) & 1ull)) s[i] = -INFINITY;
                    }
                    {   // four independent chains instead of one 64-long dependency chain
                        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                        for (int i = 0; i < AT_KPT; i += 4) {
                            mx[0] = fmaxf(mx[0], s[i]); mx[1] = fmaxf(mx[1], s[i + 1]);
                            mx[2] = fmaxf(mx[2], s[i + 2]); mx[3] = fmaxf(mx[3], s[i + 3]);
                        }
                        mt = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                    }
                    pair_max[g & 1][part][row] = mt;
                    asm volatile("bar.sync %0, %1;" ::"r"(pair_bar), "n"(32 * AT_SPLIT) : "memory");
#pragma unroll
                    for (int q = 0; q < AT_SPLIT; ++q) mt = fmaxf(mt, pair_max[g & 1][q][row]);
                    mt *= p.scale_log2;
                }
                // this tile's P buffer was last read by the P.V product of two tiles ago
                if (g > 1) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_P_FREE + (g & 1)), ((uint32_t)(g >> 1) & 1u) ^ 1u, &abort_flag, p.status));
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (group_live) {
                    float factor = 1.f;
                    if (live && mt > -INFINITY) {
                        if (m_ref == -INFINITY) m_ref = mt;
                        else if (mt > m_ref + AT_RESCALE_GAP) { factor = fast_exp2(m_ref - mt); m_ref = mt; }
                    }
                    if (g > g0 && __any_sync(0xffffffffu, factor != 1.f)) {
                        // O may only be touched once the previous P.V product has finished
                        ok = __all_sync(0xffffffffu, mbar_wait(bar(B_P_FREE + ((g - 1) & 1)), (uint32_t)((g - 1) >> 1) & 1u, &abort_flag, p.status));
                        if (!ok) break;
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        l_sum *= factor;
#pragma unroll 1
                        for (int c0 = 0; c0 < AT_KPT; c0 += 32) {
                            float o[32];
                            tmem_ld32(tmem_o + lane_addr + col0 + c0, o);
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] *= factor;
                            tmem_st32(tmem_o + lane_addr + col0 + c0, o);
                        }
                    }
                    // P = 2^(s * c - m_ref) as bf16 pairs into this tile's P buffer in TMEM (lane = row, one column
                    // per two keys); masked scores are -inf and give exactly 0.  Rows past the tree store zeros.
                    const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                    uint32_t packed[AT_KPT / 2];
                    if (live) {
                        float ls[4] = {0.f, 0.f, 0.f, 0.f};  // independent partial sums
#pragma unroll
                        for (int i = 0; i < AT_KPT; i += 4) {
                            const float a = fast_exp2(fmaf(s[i], p.scale_log2, -m_use));
                            const float b = fast_exp2(fmaf(s[i + 1], p.scale_log2, -m_use));
                            const float c = fast_exp2(fmaf(s[i + 2], p.scale_log2, -m_use));
                            const float d = fast_exp2(fmaf(s[i + 3], p.scale_log2, -m_use));
                            ls[0] += a; ls[1] += b; ls[2] += c; ls[3] += d;
                            packed[i >> 1] = pack_bf16(a, b);
                            packed[(i >> 1) + 1] = pack_bf16(c, d);
                        }
                        l_sum += (ls[0] + ls[1]) + (ls[2] + ls[3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < AT_KPT / 2; ++i) packed[i] = 0u;
                    }
                    if constexpr (AT_KPT == 64) tmem_st32u(tmem_p[g & 1] + lane_addr + (AT_KPT / 2) * part, packed);
                    else tmem_st16u(tmem_p[g & 1] + lane_addr + (AT_KPT / 2) * part, packed);
                    if constexpr (PRECISE) {
                        // lo = p - bf16(p), recomputed from the scores 32 keys at a time (keeps the register count
                        // down); every thread of the row group has its scores in registers since the exchange of
                        // the maxima, so the S buffer may be overwritten
#pragma unroll
                        for (int c0 = 0; c0 < AT_KPT; c0 += 32) {
                            uint32_t lo[16];
                            if (live) {
#pragma unroll
                                for (int i = 0; i < 32; i += 2) {
                                    const float a = fast_exp2(fmaf(s[c0 + i], p.scale_log2, -m_use));
                                    const float b = fast_exp2(fmaf(s[c0 + i + 1], p.scale_log2, -m_use));
                                    lo[i >> 1] = pack_bf16(a - bf16_round(a), b - bf16_round(b));
                                }
                            } else {
#pragma unroll
                                for (int i = 0; i < 16; ++i) lo[i] = 0u;
                            }
                            tmem_st16u(tmem_s[g & 1] + lane_addr + (AT_KPT / 2) * part + (c0 >> 1), lo);
                        }
                    }
                }
                // keys past the end of the sequence hold whatever the cache holds: clear those V rows so
                // that 0 * garbage cannot poison the product
                if (key0 + AT_KEYS > total) {
                    const int slot = (2 * g + 1) % AT_RING;
                    ok = __all_sync(0xffffffffu, mbar_wait(bar(B_KV_FULL + slot), (uint32_t)((2 * g + 1) / AT_RING) & 1u, &abort_flag, p.status));
                    if (!ok) break;
                    uint8_t* v_ptr = base_ptr + AT_TILE + slot * AT_TILE;
                    const int first_bad = max(total - key0, 0);
                    for (int i = first_bad * 8 + (int)threadIdx.x; i < AT_KEYS * 8; i += AT_SM_THREADS) {      // 16-byte chunks, both sub-tiles
                        *reinterpret_cast<uint4*>(v_ptr + i * 16) = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4*>(v_ptr + AT_SUB + i * 16) = make_uint4(0, 0, 0, 0);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the MMA reads V through the async proxy
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                mbar_arrive(bar(B_P_READY + (g & 1)));
            }
            if (!ok) break;
            // ---- epilogue of the segment
            ok = __all_sync(0xffffffffu, mbar_wait(bar(B_O_READY), (uint32_t)(e & 1), &abort_flag, p.status));
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (group_live) {
                pair_sum[e & 1][part][row] = l_sum;
                asm volatile("bar.sync %0, %1;" ::"r"(pair_bar), "n"(32 * AT_SPLIT) : "memory");
                float l_row = 0.f;
#pragma unroll
                for (int q = 0; q < AT_SPLIT; ++q) l_row += pair_sum[e & 1][q][row];     // the same order in every thread
                const bool whole_seg = (w.t == 0 && n_tiles == w.tiles);
                if (p.cluster > 1) {
                    // all products that read the ring have finished (B_O_READY), and this CTA loads nothing more
#pragma unroll 1
                    for (int c0 = 0; c0 < AT_KPT; c0 += 32) {
                        float o[32];
                        tmem_ld32(tmem_o + lane_addr + col0 + c0, o);
                        if (live) {
                            float4* dst = reinterpret_cast<float4*>(piece_o + (size_t)row * AT_PIECE_STRIDE + col0 + c0);
#pragma unroll
                            for (int i = 0; i < 8; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                        }
                    }
                    if (live && part == 0) { piece_m[row] = m_ref; piece_l[row] = l_row; }
                } else if (whole_seg) {
                    const float inv = live ? 1.f / l_row : 0.f;
                    const size_t off = ((size_t)grow * p.H + w.h) * AT_D + col0;
#pragma unroll 1
                    for (int c0 = 0; c0 < AT_KPT; c0 += 32) {
                        float o[32];
                        tmem_ld32(tmem_o + lane_addr + col0 + c0, o);
                        if (live) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] *= inv;
#pragma unroll
                            for (int ch = 0; ch < 4; ++ch)
                                store8_split(p.out + off + c0 + 8 * ch, p.out_lo ? p.out_lo + off + c0 + 8 * ch : nullptr, o + 8 * ch);
                        }
                    }
                } else {
                    float* slot = p.slots + (size_t)(w.bh + (int)blockIdx.x) * AT_SLOT_FLOATS;
#pragma unroll 1
                    for (int c0 = 0; c0 < AT_KPT; c0 += 32) {
                        float o[32];
                        tmem_ld32(tmem_o + lane_addr + col0 + c0, o);
                        if (live) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) slot[(size_t)(col0 + c0 + i) * AT_ROWS + row] = o[i];
                        }
                    }
                    if (live && part == 0) { slot[AT_D * AT_ROWS + row] = m_ref; slot[AT_D * AT_ROWS + AT_ROWS + row] = l_row; }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(bar(B_O_FREE));
            u += n_tiles;
            ++e;
        }
    }
    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (abort_flag) {                                        // let copies still in flight land before the CTA leaves
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (p.cluster > 1) {
        // Every CTA of the cluster gets here, with or without a piece, and also after a wait that gave up.
        pdl_wait();                                          // threads that had no role have not waited yet
        cluster_sync_all();                                  // all pieces are in place and visible
        const int C = p.cluster, rank = blockIdx.x % C, head = blockIdx.x / C;
        const int rows = sched.row0[1] - sched.row0[0], width = AT_D / C, groups = width / 4;
        const uint32_t m_local = smem_u32(piece_m), l_local = smem_u32(piece_l), o_local = smem_u32(piece_o);
        if (!abort_flag) {
            for (int i = threadIdx.x; i < rows * groups; i += AT_THREADS) {
                const int row = i / groups, col = rank * width + 4 * (i % groups);
                // every piece's statistics and values are requested before any is used
                float m_c[8], l_c[8], m_all = -INFINITY;
                float4 o_c[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    if (c < C) {
                        m_c[c] = ld_cluster(cluster_addr(m_local + 4u * row, c));
                        l_c[c] = ld_cluster(cluster_addr(l_local + 4u * row, c));
                        o_c[c] = ld_cluster4(cluster_addr(o_local + 4u * (uint32_t)(row * AT_PIECE_STRIDE + col), c));
                    }
                }
#pragma unroll
                for (int c = 0; c < 8; ++c) if (c < C) m_all = fmaxf(m_all, m_c[c]);
                float l_all = 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int c = 0; c < 8; ++c) {                // pieces in ascending tile order; one without keys holds no data
                    if (c >= C || m_c[c] == -INFINITY) continue;
                    const float wgt = exp2f(m_c[c] - m_all);
                    l_all = fmaf(l_c[c], wgt, l_all);
                    acc.x = fmaf(o_c[c].x, wgt, acc.x); acc.y = fmaf(o_c[c].y, wgt, acc.y);
                    acc.z = fmaf(o_c[c].z, wgt, acc.z); acc.w = fmaf(o_c[c].w, wgt, acc.w);
                }
                const float inv = 1.f / l_all;
                const size_t off = ((size_t)(sched.row0[0] + row) * p.H + head) * AT_D + col;
                store4_split(p.out + off, p.out_lo ? p.out_lo + off : nullptr, acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
            }
        }
        cluster_sync_all();                                  // nobody leaves while its piece may still be read
    }
    if (warp == AT_W_MMA)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
#ifdef TRJ_TIMELINE
    if (threadIdx.x == 0 && u_begin >= u_end) tl_slot__ = ::trj::tl::begin(TRJ_TL_ATTENTION);   // a CTA without work never stamped its release
#endif
    TRJ_TL_END(TRJ_TL_ATTENTION);
}

// Merges the pieces of every (sequence, head) that more than one CTA worked on.  One CTA per
// (sequence, head, 16-wide slice of head_dim), thread = row; pieces are taken in ascending CTA order.
constexpr int CB_COLS = 16;
__global__ void __launch_bounds__(128) tree_attention_combine_kernel(const AtParams p, int grid_main) {
    __shared__ Sched sched;
    __shared__ float stage[AT_ROWS][CB_COLS + 1];
    // the geometry (sequence lengths, row offsets) is not produced by the main kernel: work it out while that
    // kernel may still be running, and wait for its pieces only afterwards
    pdl_launch_dependents();
    if (threadIdx.x == 0) build_sched(sched, p);
    __syncthreads();
    const int bh = blockIdx.x, b = bh / p.H, h = bh % p.H, c0 = blockIdx.y * CB_COLS;
    const long long U = sched.first[p.B];
    const long long u0 = sched.first[b] + (long long)h * sched.tiles[b], u1 = u0 + sched.tiles[b];
    // CTA c of the main kernel owns units [U*c/G, U*(c+1)/G): the owner of unit u is the largest c with U*c/G <= u
    auto owner = [&](long long u) { return (int)(((u + 1) * grid_main + U - 1) / U - 1); };
    const int c_first = owner(u0), c_last = owner(u1 - 1);
    const int row = threadIdx.x, rows = p.row_off[b + 1] - p.row_off[b];
    const bool live = row < rows;
    // a CTA in between may own no unit at all (grid larger than the unit count): it wrote nothing
    auto has_piece = [&](int c) {
        const long long rb = U * c / grid_main, re = U * (c + 1) / grid_main;
        return (rb > u0 ? rb : u0) < (re < u1 ? re : u1);
    };
    pdl_wait();
    if (c_first == c_last) return;                           // written directly by its only CTA
    if (live) {
        float m_all = -INFINITY;
        for (int c = c_first; c <= c_last; ++c)
            if (has_piece(c)) m_all = fmaxf(m_all, p.slots[(size_t)(bh + c) * AT_SLOT_FLOATS + AT_D * AT_ROWS + row]);
        float l_all = 0.f, acc[CB_COLS];
#pragma unroll
        for (int i = 0; i < CB_COLS; ++i) acc[i] = 0.f;
        for (int c = c_first; c <= c_last; ++c) {
            if (!has_piece(c)) continue;
            const float* slot = p.slots + (size_t)(bh + c) * AT_SLOT_FLOATS;
            const float m = slot[AT_D * AT_ROWS + row];
            if (m == -INFINITY) continue;
            const float wgt = exp2f(m - m_all);
            l_all = fmaf(slot[AT_D * AT_ROWS + AT_ROWS + row], wgt, l_all);
#pragma unroll
            for (int i = 0; i < CB_COLS; ++i) acc[i] = fmaf(slot[(size_t)(c0 + i) * AT_ROWS + row], wgt, acc[i]);
        }
        const float inv = 1.f / l_all;
#pragma unroll
        for (int i = 0; i < CB_COLS; ++i) stage[row][i] = acc[i] * inv;
    }
    __syncthreads();
    // rows x 16 values -> each thread stores 8 consecutive values (16 bytes) of one row
    for (int i = threadIdx.x; i < rows * 2; i += 128) {
        const int r = i >> 1, q8 = (i & 1) * 8;
        const size_t off = ((size_t)(p.row_off[b] + r) * p.H + h) * AT_D + c0 + q8;
        store8_split(p.out + off, p.out_lo ? p.out_lo + off : nullptr, &stage[r][q8]);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn at_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
    });
    return fn;
}
// bf16 matrix [rows][cols] row-major, boxes of [128 rows][64 cols], 128-byte swizzle, zero fill.
bool at_make_map(CUtensorMap* map, const void* base_ptr, size_t rows, size_t cols) {
    EncodeTiledFn fn = at_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {64, 128};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base_ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int AT_MAX_GRID = 148;
constexpr int AT_WHOLE_HEAD_TILES = 8;      // up to 1024 keys: heads are handled one by one when B == 1
constexpr int AT_CLUSTER_MAX_TILES_DEFAULT = 1 << 20;

// How many CTAs may share a head (as one thread-block cluster) when every head is handled on its own: the largest
// of 4 and 2 for which all H clusters are resident at once, else 1.  Asked of the driver once per head count.
int at_cluster_size(int H) {
    static std::mutex mu;
    static int cached_h = -1, cached_c = 1;
    std::lock_guard<std::mutex> lock(mu);
    if (cached_h == H) return cached_c;
    int pick = 1;
    if (cudaFuncSetAttribute(tree_attention_tc_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AT_SMEM) == cudaSuccess) {
        for (int c = 4; c >= 2 && pick == 1; c /= 2) {
            if (H * c > AT_MAX_GRID) continue;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(H * c); cfg.blockDim = dim3(at_threads(2)); cfg.dynamicSmemBytes = AT_SMEM;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = c; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, tree_attention_tc_kernel<2, true>, &cfg) == cudaSuccess && n >= H) pick = c;
        }
    }
    (void)cudaGetLastError();                                // a refused query is not an error of the caller
    cached_h = H; cached_c = pick;
    return pick;
}

// Longest prefix (in key tiles) that is still given to clusters.  H clusters of 4 use 4 * H CTAs (128 of the 148 SMs
// for 32 heads) and need no merge kernel; the contiguous-range shape uses every SM but pays for a second kernel and
// for the pieces' round trip through memory, which only a long prefix repays.  TRJ_AT_CLUSTER_MAX_TILES overrides
// the default (a tuning knob, read once).
int at_cluster_max_tiles() {
    static const int value = [] {
        const char* e = getenv("TRJ_AT_CLUSTER_MAX_TILES");
        const int v = e ? atoi(e) : 0;
        return v > 0 ? v : AT_CLUSTER_MAX_TILES_DEFAULT;
    }();
    return value;
}

// Launch shape.  The host only knows an upper bound of the key count; CTAs whose range turns out empty do no work.
struct AtPlan { int grid, cluster; bool merge_kernel; int split; };   // split: threads per query row in the softmax
AtPlan at_plan(int32_t B, int32_t H, int32_t max_len) {
    const int tiles_bound = (max_len + AT_KEYS - 1) / AT_KEYS;
    const long long units_bound = (long long)B * H * tiles_bound;
    // One sequence: every head on its own.  A head's tiles are shared by the CTAs of a cluster, which merge their
    // pieces through distributed shared memory: no pieces go through global memory and no merge kernel is needed.
    // Where clusters do not fit, one CTA takes a whole head of up to AT_WHOLE_HEAD_TILES tiles.
    if (B == 1 && H <= AT_MAX_GRID) {
        const int c = tiles_bound >= 2 ? at_cluster_size(H) : 1;
        if ((c > 1 && tiles_bound <= at_cluster_max_tiles()) || tiles_bound <= AT_WHOLE_HEAD_TILES) return AtPlan{H * c, c, false, 2};
    }
    // contiguous ranges + merge kernel; batches of small trees leave row groups empty, so four threads share a row
    return AtPlan{(int)(units_bound < AT_MAX_GRID ? units_bound : AT_MAX_GRID), 1, true, B > 1 ? 4 : 2};
}

}  // namespace

#ifdef TRJ_TIMELINE
cudaError_t timeline_reset_attention(cudaStream_t st) { return tl::reset(st); }
int timeline_read_attention(int kind, int max_launches, uint64_t* b, uint64_t* e) { return tl::read(kind, max_launches, b, e); }
#endif

int tree_attention_grid(int32_t B, int32_t H, int32_t max_len) { return at_plan(B, H, max_len).grid; }

bool tree_attention_tc_supported(int32_t D, int32_t dtype, int32_t max_rows) {
    return D == AT_D && dtype == TRJ_BF16 && max_rows <= AT_ROWS && at_encode_fn() != nullptr;
}

// Workspace: 256-byte header (status word), then one slot per possible piece: a CTA range can start a
// new (sequence, head) at most B*H times in total and each of the <= 148 CTAs opens at most one more.
size_t tree_attention_tc_workspace(int32_t B, int32_t H) {
    return 256 + ((size_t)B * H + AT_MAX_GRID) * AT_SLOT_FLOATS * sizeof(float);
}

cudaError_t launch_tree_attention_tc(const void* q, const void* k_slab, const void* v_slab, const uint64_t* anc,
                                     int32_t anc_words, const Batch& bt, int32_t H, int32_t Hkv, int32_t max_seq, void* out,
                                     void* out_lo, void* workspace, cudaStream_t st, int* status) {
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(tree_attention_tc_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AT_SMEM);
        if (attr_err == cudaSuccess)
            attr_err = cudaFuncSetAttribute(tree_attention_tc_kernel<4, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AT_SMEM);
        if (attr_err == cudaSuccess)
            attr_err = cudaFuncSetAttribute(tree_attention_tc_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AT_SMEM);
        if (attr_err == cudaSuccess)
            attr_err = cudaFuncSetAttribute(tree_attention_tc_kernel<4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AT_SMEM);
    });
    if (attr_err != cudaSuccess) return attr_err;
    CUtensorMap map_q, map_k, map_v;
    if (!at_make_map(&map_q, q, (size_t)bt.rows_total, (size_t)H * AT_D) ||
        !at_make_map(&map_k, k_slab, (size_t)(bt.shared_cache ? 1 : bt.B) * Hkv * max_seq, AT_D) ||
        !at_make_map(&map_v, v_slab, (size_t)(bt.shared_cache ? 1 : bt.B) * Hkv * max_seq, AT_D))
        return cudaErrorInvalidValue;
    AtParams p;
    p.seq_len = bt.seq_len; p.row_off = bt.row_off; p.anc = anc; p.anc_words = anc_words;
    p.B = bt.B; p.H = H; p.max_seq = max_seq;
    p.Hkv = Hkv; p.group = H / Hkv;
    p.early_ok = bt.cached_rows_final;
    p.shared_cache = bt.shared_cache;
    p.out = (__nv_bfloat16*)out;
    p.out_lo = (__nv_bfloat16*)out_lo;
    p.status = status ? status : (int*)workspace;
    p.slots = (float*)((char*)workspace + 256);
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)AT_D);
    if ((long long)bt.B * H * ((bt.max_len + AT_KEYS - 1) / AT_KEYS) > 0x7fffffffLL) return cudaErrorInvalidValue;   // unit indices are ints
    const AtPlan plan = at_plan(bt.B, H, bt.max_len);
    p.cluster = plan.cluster;
    count_launch();
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.grid); cfg.blockDim = dim3(at_threads(plan.split)); cfg.dynamicSmemBytes = AT_SMEM; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (chain_active()) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    if (plan.cluster > 1) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = plan.cluster; attr[n_attr].val.clusterDim.y = 1; attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    cfg.attrs = attr; cfg.numAttrs = n_attr;
    // inside a decoder (the caller asks for the result as a bf16 pair) the probabilities are a bf16 pair as well
    const bool precise = out_lo != nullptr;
    cudaError_t e;
    if (plan.split == 4)
        e = precise ? cudaLaunchKernelEx(&cfg, tree_attention_tc_kernel<4, true>, map_q, map_k, map_v, p)
                    : cudaLaunchKernelEx(&cfg, tree_attention_tc_kernel<4, false>, map_q, map_k, map_v, p);
    else
        e = precise ? cudaLaunchKernelEx(&cfg, tree_attention_tc_kernel<2, true>, map_q, map_k, map_v, p)
                    : cudaLaunchKernelEx(&cfg, tree_attention_tc_kernel<2, false>, map_q, map_k, map_v, p);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess || !plan.merge_kernel) return e;
    count_launch();
    // The merge kernel's predecessor is always the kernel above, and ahead of its wait it reads only the batch
    // geometry, which was complete before that kernel could start: programmatic launch is safe outside a chain too.
    e = launch_dependent(pdl_enabled(), tree_attention_combine_kernel, dim3(bt.B * H, AT_D / CB_COLS), dim3(128), 0, st, p, plan.grid);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_tree_attention(const void* q, const void* k_slab, const void* v_slab, const uint64_t* anc,
                                  int32_t anc_words, const Batch& bt, int32_t H, int32_t Hkv, int32_t D, int32_t max_seq,
                                  int32_t dtype, void* out, void* out_lo, void* workspace, size_t workspace_bytes,
                                  cudaStream_t st, int* status) {
    if (D == AT_D && dtype == TRJ_BF16 && bt.max_rows <= AT_ROWS) {
        if (!workspace || ((uintptr_t)workspace % 256) != 0 || workspace_bytes < tree_attention_tc_workspace(bt.B, H) ||
            !tree_attention_tc_supported(D, dtype, bt.max_rows))
            return cudaErrorInvalidValue;
        return launch_tree_attention_tc(q, k_slab, v_slab, anc, anc_words, bt, H, Hkv, max_seq, out, out_lo, workspace, st, status);
    }
    return launch_tree_attention_generic(q, k_slab, v_slab, anc, anc_words, bt, H, Hkv, D, max_seq, dtype, out, out_lo, st);
}

}  // namespace trj
