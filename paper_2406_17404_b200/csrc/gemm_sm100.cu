// Projection GEMM for sm_100a: y[M][N] = (x + x_lo)[M][K] . w[N][K]^T, from a handful of tree rows to a prompt's worth.
//
// The verification step multiplies a handful of rows (tens) by every weight matrix, so the job is
// to stream the weights from HBM once, at full bandwidth.  The roles are swapped with respect to a
// usual GEMM: a CTA owns 128 weight rows (the M dimension of one tcgen05.mma, accumulator lanes in
// TMEM) and ALL activation rows are the N dimension (columns of the accumulator).  Weight tiles
// [128 x 64] and the activation tile [rows x 64] arrive by TMA into 128-byte-swizzled shared memory,
// one elected thread issues the MMAs, and the 128 threads read the accumulator back with tcgen05.ld.
// In bf16 models the activations come as a bf16 pair hi + lo (lo = rounding error of hi); the two
// halves are simply further accumulator columns that the epilogue adds, so the product keeps fp32-like
// input precision at no cost in weight traffic.  K is split across CTAs when a matrix has too few
// 128-row tiles to keep every SM loading; partial sums go to a workspace and are added in a fixed
// order, so results do not depend on scheduling.  More rows than one accumulator holds (256 columns: 256 rows, or
// 128 rows as a hi + lo pair) are cut into blocks; an item is then one weight tile x one block x one K range, and
// the blocks of a weight tile are dealt to neighbouring CTAs so that the tile is fetched from HBM once and from L2
// after that.  With 256 rows per block the kernel is a 128 x 256 x 64-per-stage tensor-core GEMM, bound by the
// tensor pipe instead of by HBM.
#include <cuda.h>
#include <cstdlib>
#include <mutex>
#include <algorithm>
#include "trj_internal.h"
#include "sm100_common.cuh"
#include "timeline.cuh"

namespace trj {
namespace {

constexpr int TC_BM = 128;            // weight rows per CTA = UMMA M
constexpr int TC_BK = 64;             // bf16 elements per stage row = one 128-byte swizzle span
constexpr int TC_THREADS = 192;           // TMA warp, MMA warp, four epilogue warps
constexpr int TC_MAX_STAGES = 8;
constexpr uint32_t TC_A_BYTES = TC_BM * TC_BK * 2;
constexpr int TC_GRID = 296;              // two persistent CTAs per SM: one's ramp and tail overlap the other's stream

struct TcParams {
    int M, N, K;
    int m_blocks;       // blocks the activation rows are cut into
    int block_rows;     // rows per block (the last block may hold fewer)
    int m_pad;          // rows of a block rounded up (8 with a lo half, else 16) = rows of the activation box
    int halves;         // 1: x only, 2: x and x_lo
    int n_mma;          // N of one product: m_pad * halves, or m_pad when the halves are summed in the accumulator; a multiple of 16
    int acc_cols;       // TMEM columns of one accumulator buffer: power of two >= max(16, n_mma); two are allocated
    TopEntry* top;      // arg-max table of the epilogue (may be null); store_y == 0: the outputs themselves are not written
    int store_y;
    int pair_sum;       // hi and lo halves of a pair are two products into ONE accumulator (see tc_plan)
    int kblocks;        // ceil(K / 64)
    int tiles, splits, stages;
    float* out;         // [splits][M][N]
    int* status;        // device word: 0, or TRJ_ETIMEOUT once a wait expired
    int self_boxes;     // [128 x 64] tiles of this projection's own weights that the early CTAs request into L2
    int ahead_boxes, ahead_kblocks, ahead_ctas;   // [128 x 64] tiles of a later projection's weights to request into L2
};

using namespace sm100;

// Persistent kernel: CTA c works on items c, c + grid, c + 2*grid, ... where an item is one 128-row weight tile
// restricted to one K range (tile = item / splits, split = item % splits).  The TMA ring runs through item
// boundaries, and the accumulator is double-buffered in TMEM so that the epilogue of one item overlaps the
// loads and MMAs of the next.  Warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: epilogue.
// TOP: the epilogue also leaves arg-max candidates (the LM head of a verification step); the plain instantiation
// carries none of that code (the epilogue's instruction schedule is on every projection's critical path).
template <bool TOP>
__global__ void __launch_bounds__(TC_THREADS, 2) gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w,
                                                                const __grid_constant__ CUtensorMap map_x,
                                                                const __grid_constant__ CUtensorMap map_xlo, const __grid_constant__ CUtensorMap map_ahead,
                                                                const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * TC_MAX_STAGES + 4];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;     // swizzled tiles need 1024-byte alignment
    const uint32_t b_bytes = (uint32_t)(p.m_pad * p.halves) * TC_BK * 2;   // activation rows of a stage: hi tile, then lo tile
    const uint32_t stage_bytes = TC_A_BYTES + b_bytes;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[TC_MAX_STAGES]);
    const uint32_t acc_full0 = smem_u32(&bars[2 * TC_MAX_STAGES]), acc_empty0 = smem_u32(&bars[2 * TC_MAX_STAGES + 2]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int per_tile = p.splits * p.m_blocks;              // items of one weight tile: block index fastest
    const int items = p.tiles * per_tile;
    TRJ_TL_DECL;
    TRJ_TL_ENTER();

    pdl_launch_dependents();
    if (threadIdx.x == 32) {                                 // have the tensor maps on their way before the first copy needs them
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_xlo) : "memory");
    }
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full0 + 8 * b, 1); mbar_init(acc_empty0 + 8 * b, 128); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {      // one warp allocates the two accumulator buffers
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)(2 * p.acc_cols)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- producer: stream weight and activation tiles, item after item.
            // Weights are constants, so the first ring-full of weight tiles is requested BEFORE waiting for the
            // previous kernel of the stream; the activation tiles of those stages follow after the wait.
            bool ok = true;
            int prefetched = 0;
            // weights that are read once go through L2 with an evict-first policy; with several row blocks they are
            // read again by the neighbouring CTAs and are left under the default policy
            const uint64_t evict_first = l2_evict_first_policy();
            uint64_t w_policy;
            asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(w_policy));
            if (p.m_blocks == 1) w_policy = evict_first;
            for (int pass = 0; pass < 2 && ok; ++pass) {
                int fill = 0;                                // running stage counter
                for (int item = blockIdx.x; item < items && ok; item += gridDim.x) {
                    const int tile = item / per_tile, split = (item % per_tile) / p.m_blocks;
                    const int row0 = ((item % per_tile) % p.m_blocks) * p.block_rows;
                    const int kb0 = (int)((long long)split * p.kblocks / p.splits);
                    const int kb1 = (int)((long long)(split + 1) * p.kblocks / p.splits);
                    for (int kb = kb0; kb < kb1; ++kb, ++fill) {
                        const int s = fill % p.stages;
                        const uint32_t a_dst = tiles_base + s * stage_bytes, b_dst = a_dst + TC_A_BYTES;
                        const uint32_t bar = full0 + 8 * s;
                        if (pass == 0) {                     // weights only, at most one ring-full
                            if (fill >= p.stages) break;
                            mbar_expect_tx(bar, stage_bytes);
                            tma_load_2d_hint(a_dst, &map_w, kb * TC_BK, tile * TC_BM, bar, w_policy);
                            prefetched = fill + 1;
                            continue;
                        }
                        if (fill >= prefetched) {
                            const uint32_t phase = (uint32_t)(fill / p.stages) & 1u;
                            ok = mbar_wait(empty0 + 8 * s, phase ^ 1u, &abort_flag, p.status);
                            if (!ok) break;
                            mbar_expect_tx(bar, stage_bytes);
                            tma_load_2d_hint(a_dst, &map_w, kb * TC_BK, tile * TC_BM, bar, w_policy);
                        }
                        tma_load_2d(b_dst, &map_x, kb * TC_BK, row0, bar);
                        if (p.halves == 2) tma_load_2d(b_dst + (uint32_t)p.m_pad * TC_BK * 2, &map_xlo, kb * TC_BK, row0, bar);
                    }
                    if (pass == 0 && fill >= p.stages) break;
                }
                if (pass == 0) {
                    // CTAs that run while the previous kernel still does: a later projection's weights into L2
                    if ((int)blockIdx.x < p.ahead_ctas) {
                        for (int i = blockIdx.x; i < p.self_boxes; i += p.ahead_ctas)      // this projection's own weights first
                            tma_prefetch_l2_2d(&map_w, (i % p.kblocks) * TC_BK, (i / p.kblocks) * TC_BM);
                        for (int i = blockIdx.x; i < p.ahead_boxes; i += p.ahead_ctas)
                            tma_prefetch_l2_2d(&map_ahead, (i % p.ahead_kblocks) * TC_BK, (i / p.ahead_kblocks) * TC_BM);
                    }
                    pdl_wait();                              // activations come from the previous kernel
                    TRJ_TL_BEGIN(TRJ_TL_GEMM);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer
            const uint32_t idesc = idesc_bf16(TC_BM, p.n_mma);
            int fill = 0, j = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < items && ok; item += gridDim.x, ++j) {
                const int split = (item % per_tile) / p.m_blocks;
                const int nkb = (int)((long long)(split + 1) * p.kblocks / p.splits) - (int)((long long)split * p.kblocks / p.splits);
                const int buf = j & 1;
                // the epilogue must have drained this accumulator buffer (two items ago)
                ok = mbar_wait(acc_empty0 + 8 * buf, ((uint32_t)(j >> 1) & 1u) ^ 1u, &abort_flag, p.status);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * p.acc_cols);
                for (int i = 0; i < nkb && ok; ++i, ++fill) {
                    const int s = fill % p.stages;
                    const uint32_t phase = (uint32_t)(fill / p.stages) & 1u;
                    ok = mbar_wait(full0 + 8 * s, phase, &abort_flag, p.status);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_addr = tiles_base + s * stage_bytes;
                    const uint64_t a_desc = desc_kmajor_sw128(a_addr), b_desc = desc_kmajor_sw128(a_addr + TC_A_BYTES);
                    if (!p.pair_sum) {
#pragma unroll
                        for (int kk = 0; kk < TC_BK / 16; ++kk)  // 16 bf16 = 32 bytes = 2 descriptor units per MMA
                            umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (i > 0 || kk > 0) ? 1u : 0u);
                    } else {
                        // the low halves' tile lies m_pad rows of 128 bytes behind the high halves' tile
                        const uint64_t lo_desc = desc_kmajor_sw128(a_addr + TC_A_BYTES + (uint32_t)p.m_pad * TC_BK * 2);
#pragma unroll
                        for (int kk = 0; kk < TC_BK / 16; ++kk) {
                            umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (i > 0 || kk > 0) ? 1u : 0u);
                            umma_bf16(d_tmem, a_desc + 2 * kk, lo_desc + 2 * kk, idesc, 1u);
                        }
                    }
                    umma_commit(empty0 + 8 * s);             // frees the stage once these MMAs have read it
                }
                if (ok) umma_commit(acc_full0 + 8 * buf);    // accumulator of this item complete
            }
        }
    } else {
        // ---------------- epilogue: lane = weight row, columns = activation rows (hi half, then lo half)
        const int q = warp & 3;                              // TMEM lane group this warp may access
        int j = 0;
        bool ok = true;
        pdl_wait();                                          // the output buffer may still be read by the previous kernel
        for (int item = blockIdx.x; item < items && ok; item += gridDim.x, ++j) {
            const int tile = item / per_tile, split = (item % per_tile) / p.m_blocks;
            const int row0 = ((item % per_tile) % p.m_blocks) * p.block_rows;
            const int buf = j & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(acc_full0 + 8 * buf, (uint32_t)(j >> 1) & 1u, &abort_flag, p.status));
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int n = tile * TC_BM + q * 32 + lane;
            const uint32_t taddr = tmem_base + (uint32_t)(buf * p.acc_cols) + ((uint32_t)(q * 32) << 16);
            float* out = p.out + (size_t)split * p.M * p.N;
            // eight columns (activation rows) of each half per round trip: measured faster than 16 or 32 at a time
            for (int c0 = 0; c0 < p.m_pad; c0 += 8) {
                float hi[8], lo[8];
                tmem_ld8(taddr + c0, hi);
                const bool two_halves = p.halves == 2 && !p.pair_sum;
                if (two_halves) tmem_ld8(taddr + p.m_pad + c0, lo);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (!TOP || p.store_y) {
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj) {
                        const int m = row0 + c0 + jj;
                        if (c0 + jj < p.block_rows && m < p.M && n < p.N) out[(size_t)m * p.N + n] = two_halves ? hi[jj] + lo[jj] : hi[jj];
                    }
                }
                if constexpr (TOP) {
                    if (two_halves) {
#pragma unroll
                        for (int jj = 0; jj < 8; ++jj) hi[jj] += lo[jj];
                    }
                    // this warp's 32 outputs of every row: best value, its index (ties: the smaller index), runner-up
                    float v1[8], v2[8];
                    int i1[8];
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj) { v1[jj] = n < p.N ? hi[jj] : -INFINITY; i1[jj] = n < p.N ? n : 0x7fffffff; v2[jj] = -INFINITY; }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                        for (int jj = 0; jj < 8; ++jj) {
                            const float ov1 = __shfl_xor_sync(0xffffffffu, v1[jj], o), ov2 = __shfl_xor_sync(0xffffffffu, v2[jj], o);
                            const int oi1 = __shfl_xor_sync(0xffffffffu, i1[jj], o);
                            const bool mine = v1[jj] > ov1 || (v1[jj] == ov1 && i1[jj] < oi1);
                            v2[jj] = fmaxf(mine ? ov1 : v1[jj], fmaxf(v2[jj], ov2));
                            v1[jj] = mine ? v1[jj] : ov1;
                            i1[jj] = mine ? i1[jj] : oi1;
                        }
                    }
                    if (lane == 0) {
#pragma unroll
                        for (int jj = 0; jj < 8; ++jj) {
                            const int m = row0 + c0 + jj;
                            if (c0 + jj < p.block_rows && m < p.M)
                                p.top[((size_t)m * p.tiles + tile) * 4 + q] = TopEntry{v1[jj], i1[jj], v2[jj]};
                        }
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(acc_empty0 + 8 * buf);
        }
    }
    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (abort_flag) {                                        // let copies that are still in flight land before the CTA leaves
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)(2 * p.acc_cols)) : "memory");
    TRJ_TL_END(TRJ_TL_GEMM);
    TRJ_TL_LEAVE();
}

// y[i] = sum_s part[s][i], fixed order.
__global__ void reduce_splits_kernel(const float4* __restrict__ part, float4* __restrict__ y, size_t n4, int splits) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        float4 a = part[i];
        for (int s = 1; s < splits; ++s) {
            const float4 b = part[(size_t)s * n4 + i];
            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        }
        y[i] = a;
    }
}

// Self-test of the time-out path: one thread waits, with the given poll limit, on a barrier that nobody ever
// arrives at.  The wait is the very function the projection and attention kernels use; it gives up, leaves
// TRJ_ETIMEOUT in *status and the kernel returns normally.
__global__ void wait_expiry_selftest_kernel(int* status, uint32_t polls) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        (void)mbar_wait(smem_u32(&bar), 0u, &abort_flag, status, polls);
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

// bf16 matrix [rows][K] row-major -> tiles of [box_rows][64] with 128-byte swizzle, zero fill out of range.
bool make_map(CUtensorMap* map, const void* base, int rows, int K, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int round_up(int x, int a) { return (x + a - 1) / a * a; }

}  // namespace

bool gemm_tc_supported(const void* x, const void* x_lo, const void* w, const float* y, int32_t M, int32_t N, int32_t K,
                       int32_t dtype) {
    if (dtype != TRJ_BF16 || M < 1 || K < TC_BK || K % 8 != 0 || N < 4 || N % 4 != 0) return false;
    if (((uintptr_t)x | (uintptr_t)x_lo | (uintptr_t)w | (uintptr_t)y) % 16 != 0) return false;
    return encode_fn() != nullptr;
}

namespace {

// Launch geometry of one projection.
struct TcPlan {
    int halves, m_blocks, block_rows, m_pad, n_mma, acc_cols, stages, grid_cap, tiles, kblocks, splits, pair_sum;
    size_t stage_bytes;
};

// Number of K ranges per weight tile.  Items (tiles x row blocks x splits) are dealt round-robin to a grid of at
// most grid_cap CTAs, so the choice trades balance (items close to a multiple of the grid) against the extra
// traffic of the partial sums, about 2*splits*M/K of the weight bytes (weighted, see below).  When no consumer kernel adds the pieces
// (`finished`: the caller wants y itself) a reduce kernel has to read them again and is one more launch: then a
// single K range is taken as soon as the tiles alone fill most of the grid.
int tc_splits(int M, int K, int units, int kblocks, int grid_cap, bool finished) {
    if (finished && units * 5 >= grid_cap * 4) return 1;
    int best = 1;
    double best_score = 0.0;
    // A split that leaves a good part of the grid without any item is only taken when no split fills it: 224 long
    // items on 296 CTAs (gate/up of the LLaMA-3 shape as one K range) scored like five K ranges but ran 2 % slower.
    bool can_fill = false;
    for (int s = 1; s <= 16 && s <= (kblocks >= 4 ? kblocks / 4 : 1); ++s) can_fill |= units * s * 20 >= grid_cap * 19;
    for (int s = 1; s <= 16 && s <= (kblocks >= 4 ? kblocks / 4 : 1); ++s) {
        const int items = units * s, rounds = (items + grid_cap - 1) / grid_cap;
        if (can_fill && items * 20 < grid_cap * 19) continue;
        const double balance = (double)items / ((double)rounds * grid_cap);
        // the pieces cost more than their own bytes: the consumer kernel that adds them sits between two projections,
        // where nothing hides it (weight 4 measured on the 7B step: gate/up goes from 5 to 3 pieces, 3.415 -> 3.393 ms;
        // weights 8 and 16 choose the same splits)
        const double score = balance / (1.0 + 4.0 * 2.0 * s * M / K);
        if (score > best_score * 1.02) { best_score = score; best = s; }      // prefer fewer splits on near ties
    }
    return best;
}

TcPlan tc_plan(int M, int N, int K, int halves, bool finished) {
    TcPlan pl;
    pl.halves = halves;
    // an accumulator buffer holds 256 columns: 256 rows, or 128 rows as a hi + lo pair
    const int max_rows = halves == 2 ? 128 : 256, quantum = halves == 2 ? 8 : 16;
    pl.m_blocks = (M + max_rows - 1) / max_rows;
    // A pair normally rides in one product whose accumulator holds the hi columns, then the lo columns, which the
    // epilogue adds.  For 65-128 rows that accumulator would take 256 columns a buffer and leave room for one CTA per
    // SM only; there the two halves are two products into the same 128 columns instead (twice the instructions and
    // twice the shared-memory reads of the weight tile).
    // Only where it buys the second CTA (three stages of both must fit: up to 80 rows); with one CTA per SM either
    // way the single product is faster (96 rows: 4.9 against 5.8 ms per 7B step).
    pl.pair_sum = (halves == 2 && pl.m_blocks == 1 && M > 64 &&
                   3 * (TC_A_BYTES + (size_t)round_up(M, 16) * 2 * TC_BK * 2) <= 108 * 1024) ? 1 : 0;
    pl.block_rows = round_up((M + pl.m_blocks - 1) / pl.m_blocks, pl.pair_sum ? 16 : quantum);   // the lo box must start on a 1024-byte boundary: 8 rows
    pl.m_pad = pl.block_rows;
    pl.n_mma = pl.pair_sum ? pl.m_pad : pl.m_pad * halves;
    // the epilogue reads 8 columns at a time from each half, so a buffer must cover the last such read
    const int reach = (halves == 2 && !pl.pair_sum ? pl.m_pad : 0) + round_up(pl.m_pad, 16);
    pl.acc_cols = 16;
    while (pl.acc_cols < reach) pl.acc_cols *= 2;
    pl.kblocks = (K + TC_BK - 1) / TC_BK;      // a ragged last block reads zeros past K (both operands)
    pl.tiles = (N + TC_BM - 1) / TC_BM;
    pl.stage_bytes = TC_A_BYTES + (size_t)pl.m_pad * halves * TC_BK * 2;
    // Two CTAs per SM (one's ramp and drain overlap the other's stream) when both fit: at least three stages in
    // ~108 KB each and both pairs of accumulator buffers in the 512 columns of tensor memory.  Otherwise one CTA
    // per SM with as deep a ring as shared memory allows.
    const bool two_per_sm = 2 * pl.acc_cols <= 256 && 3 * pl.stage_bytes <= 108 * 1024;
    if (two_per_sm) {
        pl.stages = (int)std::min<size_t>(4, (108 * 1024) / pl.stage_bytes);
        pl.grid_cap = TC_GRID;
    } else {
        pl.stages = (int)std::min<size_t>(6, (216 * 1024) / pl.stage_bytes);
        pl.grid_cap = TC_GRID / 2;
    }
    pl.splits = tc_splits(M, K, pl.tiles * pl.m_blocks, pl.kblocks, pl.grid_cap, finished);
    return pl;
}

}  // namespace

// Workspace: a 256-byte header whose first word is the device status, then the split-K partial sums.
size_t gemm_tc_workspace(int32_t M, int32_t N, int32_t K) {
    if (K % 8 != 0 || K < TC_BK || M < 1) return 256;
    int s = 1;
    for (int halves = 1; halves <= 2; ++halves)
        for (int finished = 0; finished <= 1; ++finished) s = std::max(s, tc_plan(M, N, K, halves, finished != 0).splits);
    return 256 + (s > 1 ? align_up((size_t)s * M * N * sizeof(float), 256) : 0);
}

cudaError_t launch_gemm_tc(const void* x, const void* x_lo, const void* w, float* y, int32_t M, int32_t N, int32_t K,
                           void* workspace, cudaStream_t st, Parts* parts, const WeightPrefetch* ahead, int* status,
                           const TopTable* top) {
    if (!status) status = (int*)workspace;
    workspace = (char*)workspace + 256;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(gemm_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        if (attr_err == cudaSuccess)
            attr_err = cudaFuncSetAttribute(gemm_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
    });
    if (attr_err != cudaSuccess) return attr_err;
    const TcPlan pl = tc_plan(M, N, K, x_lo ? 2 : 1, parts == nullptr);
    if (pl.stages < 2) return cudaErrorInvalidConfiguration;
    TcParams p;
    p.M = M; p.N = N; p.K = K;
    p.halves = pl.halves; p.m_blocks = pl.m_blocks; p.block_rows = pl.block_rows; p.m_pad = pl.m_pad;
    p.n_mma = pl.n_mma; p.acc_cols = pl.acc_cols; p.kblocks = pl.kblocks; p.tiles = pl.tiles; p.pair_sum = pl.pair_sum;
    p.splits = pl.splits; p.stages = pl.stages;
    p.top = nullptr; p.store_y = 1;
    if (top) {                                               // the accumulator must hold finished sums of all rows
        if (!top->entries || parts || pl.splits != 1 || pl.m_blocks != 1) return cudaErrorInvalidValue;
        p.top = top->entries; p.store_y = top->store_y;
    }
    p.out = p.splits > 1 ? (float*)workspace : y;
    p.status = status;
    CUtensorMap map_w, map_x, map_xlo, map_ahead;
    p.ahead_boxes = 0; p.ahead_kblocks = 1; p.ahead_ctas = 0; p.self_boxes = 0;
    const bool want_ahead = ahead && ahead->ctas > 0 && ahead->w && ahead->K % 8 == 0 && ahead->K >= TC_BK &&
                            ((uintptr_t)ahead->w % 16) == 0;
    if (want_ahead) {
        if (!make_map(&map_ahead, ahead->w, ahead->N, ahead->K, TC_BM)) return cudaErrorInvalidValue;
        const size_t all = (size_t)((ahead->N + TC_BM - 1) / TC_BM) * ((ahead->K + TC_BK - 1) / TC_BK);
        const size_t asked = ahead->bytes / TC_A_BYTES;
        p.ahead_kblocks = (ahead->K + TC_BK - 1) / TC_BK;
        p.ahead_boxes = (int)(asked < all ? asked : all);
        p.ahead_ctas = ahead->ctas;
        const size_t own = (size_t)pl.tiles * pl.kblocks, want_self = ahead->self_bytes / TC_A_BYTES;
        p.self_boxes = (int)(want_self < own ? want_self : own);
    }
    if (!make_map(&map_w, w, N, K, TC_BM) || !make_map(&map_x, x, M, K, p.m_pad) ||
        !make_map(&map_xlo, x_lo ? x_lo : x, M, K, p.m_pad))
        return cudaErrorInvalidValue;
    if (!want_ahead) map_ahead = map_w;                      // never used: no CTA asks
    count_launch();
    const int items = p.tiles * p.m_blocks * p.splits;
    cudaError_t e = launch_chain(p.top ? gemm_tc_kernel<true> : gemm_tc_kernel<false>, dim3(items < pl.grid_cap ? items : pl.grid_cap),
                                 dim3(TC_THREADS), p.stages * pl.stage_bytes + 1024, st, map_w, map_x, map_xlo, map_ahead, p);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (parts) *parts = Parts{p.out, p.splits, (size_t)M * N};
    if (e != cudaSuccess || p.splits == 1 || parts) return e;
    count_launch();
    const size_t n4 = (size_t)M * N / 4;           // N % 4 == 0 is part of gemm_tc_supported
    reduce_splits_kernel<<<(unsigned)((n4 + 255) / 256 < 592 ? (n4 + 255) / 256 : 592), 256, 0, st>>>(
        (const float4*)workspace, (float4*)y, n4, p.splits);
    return cudaGetLastError();
}

#ifdef TRJ_TIMELINE
cudaError_t timeline_reset_gemm(cudaStream_t st) { return tl::reset(st); }
int timeline_read_gemm(int kind, int max_launches, uint64_t* b, uint64_t* e) { return tl::read(kind, max_launches, b, e); }
int timeline_gemm_ctas_per_sm() { return tl::sm_peak(); }
#endif

cudaError_t launch_wait_expiry_selftest(int* status, uint32_t polls, cudaStream_t st) {
    count_launch();
    wait_expiry_selftest_kernel<<<1, 32, 0, st>>>(status, polls);
    return cudaGetLastError();
}

bool gemm_top_table_ok(int32_t M, int32_t N, int32_t K, int32_t dtype, bool pair) {
    if (!gemm_tc_shape(M, N, K, dtype)) return false;
    const TcPlan pl = tc_plan(M, N, K, pair ? 2 : 1, true);
    return pl.splits == 1 && pl.m_blocks == 1 && pl.stages >= 2;
}

bool gemm_tc_shape(int32_t M, int32_t N, int32_t K, int32_t dtype) {
    return dtype == TRJ_BF16 && M >= 1 && K >= TC_BK && K % 8 == 0 && N >= 4 && N % 4 == 0;
}

cudaError_t launch_gemm(const void* x, const void* x_lo, const void* w, float* y, int32_t M, int32_t N, int32_t K,
                        int32_t dtype, void* workspace, size_t workspace_bytes, cudaStream_t st, Parts* parts,
                        const WeightPrefetch* ahead, int* status, const TopTable* top) {
    if (gemm_tc_shape(M, N, K, dtype)) {
        if (!workspace || workspace_bytes < gemm_tc_workspace(M, N, K) || ((uintptr_t)workspace % 256) != 0 ||
            !gemm_tc_supported(x, x_lo, w, y, M, N, K, dtype))
            return cudaErrorInvalidValue;
        return launch_gemm_tc(x, x_lo, w, y, M, N, K, workspace, st, parts, ahead, status, top);
    }
    if (top) return cudaErrorInvalidValue;                   // the caller asks gemm_top_table_ok first
    if (parts) *parts = whole(y);
    return launch_gemm_simt(x, x_lo, w, y, M, N, K, dtype, st);
}

}  // namespace trj
