// Projection with its consumer folded in, for the two places of a decoder layer where the consumer is a pure
// element-wise map of a weight tile's finished values: QKV projection -> rotary embedding + K/V append, and
// gate/up projection -> SwiGLU.
//
// The plain projection kernel (gemm_sm100.cu) cuts K into ranges to keep every SM loading and leaves the ranges'
// partial sums in global memory for a separate kernel to add.  Here the K ranges of one weight tile are the CTAs of
// one thread-block cluster, working on the same tile at the same time.  Every CTA puts its partial accumulator
// (128 weight rows x the activation rows, fp32) into its own shared memory, and after a cluster-wide hand-shake each
// CTA adds up, in a fixed order, a share of the activation rows from all partials through distributed shared memory
// and applies the consumer to the finished values: no partial sums in global memory, no second kernel.
//   * QKV: a 128-row weight tile is exactly one head of q, k or v, so the rotation partners (i, i + 64) are in the
//     tile; q goes to the q buffer, k and v to their cache rows.
//   * gate/up: a tile is 64 gate rows plus the 64 up rows of the same features (two TMA boxes), so silu(g) * u is in
//     the tile; the result is written as the bf16 pair the down projection takes.
// Mainloop, roles and barriers are those of the plain kernel (TMA ring, one MMA-issuing thread, accumulator
// double-buffered in tensor memory).  Every wait is bounded, including the cluster hand-shake.
#include <cuda.h>
#include <algorithm>
#include <mutex>
#include "trj_internal.h"
#include "sm100_common.cuh"
#include "timeline.cuh"

namespace trj {
namespace {

using namespace sm100;

constexpr int FU_BM = 128;                // weight rows per tile = UMMA M
constexpr int FU_BK = 64;
constexpr int FU_THREADS = 192;           // TMA warp, MMA warp, four epilogue warps
constexpr int FU_MAX_STAGES = 4;
constexpr int FU_MAX_CLUSTER = 8;
constexpr uint32_t FU_A_BYTES = FU_BM * FU_BK * 2;
constexpr int FU_CTAS = 296;              // two CTAs per SM

enum { FU_ROPE = 0, FU_SWIGLU = 1 };

struct FuParams {
    int mode;
    int M, N, K;                // activation rows, weight rows of the matrix, contraction length
    int m_pad, n_mma, acc_cols, kblocks, tiles, stages, cluster;
    int pair_offset;            // SwiGLU: row distance between a gate row and its up row (d_ff); RoPE: unused
    int* status;
    // RoPE: q -> q_out [rows][H][D]; k, v -> cache rows of the layer slab [B][Hkv][max_seq][D]
    const double* inv_freq; const int32_t* depth; const int32_t* seq_len; const int32_t* row_off;
    int B, H, Hkv, max_seq;
    __nv_bfloat16* q_out; __nv_bfloat16* k_slab; __nv_bfloat16* v_slab;
    // SwiGLU: act, act_lo [rows][f]
    __nv_bfloat16* act; __nv_bfloat16* act_lo; int f;
};

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ float ld_dsmem(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void remote_arrive(uint32_t cluster_bar_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar_addr) : "memory");
}
__device__ __forceinline__ bool try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait on a barrier that CTAs of the cluster arrive at.
__device__ __forceinline__ bool wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
    for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
        if (try_wait_cluster(bar, parity)) return true;
        if (i > 32) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    *abort_flag = 1;
    atomicExch(status, (int)TRJ_ETIMEOUT);
    return false;
}
// Barrier of the 128 epilogue threads that also tells every one of them whether any of them failed: after a wait
// that gave up, all four warps leave the tile loop together and none is left behind at a barrier.
__device__ __forceinline__ bool epilogue_barrier_any(bool failed) {
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, 1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(r) : "r"((uint32_t)failed) : "memory");
    return r != 0;
}

// Grid = clusters x cluster size.  Cluster c works on weight tiles c, c + clusters, ...; CTA rank r of a cluster
// takes K range r of every one of them.
__global__ void __launch_bounds__(FU_THREADS, 2) gemm_fused_kernel(const __grid_constant__ CUtensorMap map_w,
                                                                   const __grid_constant__ CUtensorMap map_x,
                                                                   const __grid_constant__ CUtensorMap map_xlo,
                                                                   const FuParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * FU_MAX_STAGES + 4 + 2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t b_bytes = (uint32_t)p.n_mma * FU_BK * 2;
    const uint32_t stage_bytes = FU_A_BYTES + b_bytes;
    const uint32_t staging = tiles_base + (uint32_t)p.stages * stage_bytes;        // fp32 [m_pad][128]: column-major partial
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[FU_MAX_STAGES]);
    const uint32_t acc_full0 = smem_u32(&bars[2 * FU_MAX_STAGES]), acc_empty0 = smem_u32(&bars[2 * FU_MAX_STAGES + 2]);
    const uint32_t stg_full = smem_u32(&bars[2 * FU_MAX_STAGES + 4]);              // every CTA's partial of this tile is staged
    const uint32_t stg_free = smem_u32(&bars[2 * FU_MAX_STAGES + 5]);              // every CTA is done reading this CTA's partial
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int C = p.cluster;
    const int rank = (int)cluster_rank();
    const int cluster_id = (int)blockIdx.x / C, n_clusters = (int)gridDim.x / C;
    const int kb0 = (int)((long long)rank * p.kblocks / C), kb1 = (int)((long long)(rank + 1) * p.kblocks / C);
    TRJ_TL_DECL;
    TRJ_TL_ENTER();

    pdl_launch_dependents();
    if (threadIdx.x == 32) {
        prefetch_tensormap(&map_w); prefetch_tensormap(&map_x); prefetch_tensormap(&map_xlo);
    }
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full0 + 8 * b, 1); mbar_init(acc_empty0 + 8 * b, 128); }
        mbar_init(stg_full, (uint32_t)C);
        mbar_init(stg_free, (uint32_t)C);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)(2 * p.acc_cols));
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // nobody may signal a peer's barrier before that peer has initialised it
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;

    // rows of the weight matrix that the two 64-row halves of tile t start at
    auto tile_row = [&](int t, int half) { return p.mode == FU_SWIGLU ? t * 64 + half * p.pair_offset : t * FU_BM + half * 64; };

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- producer
            bool ok = true;
            int prefetched = 0;
            const uint64_t w_policy = l2_evict_first_policy();
            for (int pass = 0; pass < 2 && ok; ++pass) {
                int fill = 0;
                for (int tile = cluster_id; tile < p.tiles && ok; tile += n_clusters) {
                    for (int kb = kb0; kb < kb1; ++kb, ++fill) {
                        const int s = fill % p.stages;
                        const uint32_t a_dst = tiles_base + s * stage_bytes, b_dst = a_dst + FU_A_BYTES;
                        const uint32_t bar = full0 + 8 * s;
                        auto load_weights = [&]() {
                            mbar_expect_tx(bar, stage_bytes);
                            tma_load_2d_hint(a_dst, &map_w, kb * FU_BK, tile_row(tile, 0), bar, w_policy);
                            tma_load_2d_hint(a_dst + FU_A_BYTES / 2, &map_w, kb * FU_BK, tile_row(tile, 1), bar, w_policy);
                        };
                        if (pass == 0) {                     // weights only, at most one ring-full, before the wait for the previous kernel
                            if (fill >= p.stages) break;
                            load_weights();
                            prefetched = fill + 1;
                            continue;
                        }
                        if (fill >= prefetched) {
                            const uint32_t phase = (uint32_t)(fill / p.stages) & 1u;
                            ok = mbar_wait(empty0 + 8 * s, phase ^ 1u, &abort_flag, p.status);
                            if (!ok) break;
                            load_weights();
                        }
                        tma_load_2d(b_dst, &map_x, kb * FU_BK, 0, bar);
                        tma_load_2d(b_dst + (uint32_t)p.m_pad * FU_BK * 2, &map_xlo, kb * FU_BK, 0, bar);
                    }
                    if (pass == 0 && fill >= p.stages) break;
                }
                if (pass == 0) { pdl_wait(); TRJ_TL_BEGIN(TRJ_TL_GEMM); }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer
            const uint32_t idesc = idesc_bf16(FU_BM, p.n_mma);
            int fill = 0, j = 0;
            bool ok = true;
            for (int tile = cluster_id; tile < p.tiles && ok; tile += n_clusters, ++j) {
                const int buf = j & 1;
                ok = mbar_wait(acc_empty0 + 8 * buf, ((uint32_t)(j >> 1) & 1u) ^ 1u, &abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * p.acc_cols);
                for (int i = 0; i < kb1 - kb0 && ok; ++i, ++fill) {
                    const int s = fill % p.stages;
                    ok = mbar_wait(full0 + 8 * s, (uint32_t)(fill / p.stages) & 1u, &abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = tiles_base + s * stage_bytes;
                    const uint64_t a_desc = desc_kmajor_sw128(a_addr), b_desc = desc_kmajor_sw128(a_addr + FU_A_BYTES);
#pragma unroll
                    for (int kk = 0; kk < FU_BK / 16; ++kk)
                        umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (i > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(empty0 + 8 * s);
                }
                if (ok) umma_commit(acc_full0 + 8 * buf);
            }
        }
    } else {
        // ---------------- epilogue: thread = weight row of the tile (TMEM lane)
        const int q = warp & 3, row_in_tile = q * 32 + lane;
        const int et = row_in_tile;                          // 0..127 among the epilogue threads
        int j = 0;
        bool ok = true;
        pdl_wait();                                          // what is written below may still be read by earlier kernels
        for (int tile = cluster_id; tile < p.tiles; tile += n_clusters, ++j) {
            const int buf = j & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(acc_full0 + 8 * buf, (uint32_t)(j >> 1) & 1u, &abort_flag, p.status));
            // the previous tile's partial must have been read by every CTA before it is overwritten
            if (ok && j > 0) ok = __all_sync(0xffffffffu, wait_cluster(stg_free, (uint32_t)(j - 1) & 1u, &abort_flag, p.status));
            if (ok) {
                tc_fence_after();
                const uint32_t taddr = tmem_base + (uint32_t)(buf * p.acc_cols) + ((uint32_t)(q * 32) << 16);
                for (int c0 = 0; c0 < p.m_pad; c0 += 8) {
                    float hi[8], lo[8];
                    tmem_ld8(taddr + c0, hi);
                    tmem_ld8(taddr + p.m_pad + c0, lo);
                    tmem_wait_ld();
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj)
                        asm volatile("st.shared.f32 [%0], %1;" ::"r"(staging + 4u * (uint32_t)((c0 + jj) * FU_BM + row_in_tile)), "f"(hi[jj] + lo[jj]) : "memory");
                }
                tc_fence_before();
                mbar_arrive(acc_empty0 + 8 * buf);           // the accumulator buffer may be refilled
            }
            if (epilogue_barrier_any(!ok)) break;            // the four epilogue warps: the whole partial is staged
            if (et < C) remote_arrive(map_to_rank(stg_full, (uint32_t)et));          // tell every CTA of the cluster (release)
            ok = __all_sync(0xffffffffu, wait_cluster(stg_full, (uint32_t)j & 1u, &abort_flag, p.status));
            if (ok) {
            // ---- this CTA finishes activation rows rank, rank + C, ...: sum of all partials in rank order, then the consumer
            if (p.mode == FU_SWIGLU) {
                // threads 0..63: feature et of the tile for rows m; threads 64..127: the same features for rows m + C
                const int feat = et & 63, sub = et >> 6;
                for (int m = rank + sub * C; m < p.M; m += 2 * C) {
                    float g = 0.f, u = 0.f;
                    for (int c = 0; c < C; ++c) {
                        const uint32_t base = map_to_rank(staging + 4u * (uint32_t)(m * FU_BM), (uint32_t)c);
                        g += ld_dsmem(base + 4u * (uint32_t)feat);
                        u += ld_dsmem(base + 4u * (uint32_t)(feat + 64));
                    }
                    const float a = g / (1.f + expf(-g)) * u;
                    const __nv_bfloat16 h = __float2bfloat16_rn(a);
                    const size_t at = (size_t)m * p.f + (size_t)tile * 64 + feat;
                    p.act[at] = h;
                    p.act_lo[at] = __float2bfloat16_rn(a - __bfloat162float(h));
                }
            } else {
                // tile = one head of q (tile < H), k (< H + Hkv) or v; thread = output dimension of the head
                const int kind = tile < p.H ? 0 : (tile < p.H + p.Hkv ? 1 : 2);
                const int head = kind == 0 ? tile : (kind == 1 ? tile - p.H : tile - p.H - p.Hkv);
                const int dim = et, fi = et & 63, partner = et ^ 64;
                const double freq = p.inv_freq[fi];
                for (int m = rank; m < p.M; m += C) {
                    float own = 0.f, other = 0.f;
                    for (int c = 0; c < C; ++c) {
                        const uint32_t base = map_to_rank(staging + 4u * (uint32_t)(m * FU_BM), (uint32_t)c);
                        own += ld_dsmem(base + 4u * (uint32_t)dim);
                        other += ld_dsmem(base + 4u * (uint32_t)partner);
                    }
                    int b = 0;
                    while (b + 1 < p.B && m >= p.row_off[b + 1]) ++b;
                    const int S = p.seq_len[b], local = m - p.row_off[b];
                    float out = own;
                    if (kind != 2) {
                        // angle in fp64 (positions reach thousands of radians), reduced to [-pi, pi] there
                        const double ang = (double)(S + p.depth[m]) * freq;
                        const double red = ang - 6.283185307179586476925 * rint(ang * 0.15915494309189533577);
                        float sn, cs;
                        sincosf((float)red, &sn, &cs);
                        out = dim < 64 ? own * cs - other * sn : own * cs + other * sn;
                    }
                    if (kind == 0) p.q_out[((size_t)m * p.H + head) * FU_BM + dim] = __float2bfloat16_rn(out);
                    else {
                        __nv_bfloat16* slab = kind == 1 ? p.k_slab : p.v_slab;
                        slab[(((size_t)b * p.Hkv + head) * p.max_seq + S + local) * FU_BM + dim] = __float2bfloat16_rn(out);
                    }
                }
            }
            }
            if (epilogue_barrier_any(!ok)) break;            // all four warps are done reading the partials
            if (et < C) remote_arrive(map_to_rank(stg_free, (uint32_t)et));
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (abort_flag) {                                        // let copies that are still in flight land before the CTA leaves
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        __syncthreads();
    }
    // nobody leaves while a peer may still read its partial or signal its barriers
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)(2 * p.acc_cols));
    TRJ_TL_END(TRJ_TL_GEMM);
    TRJ_TL_LEAVE();
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn fu_encode_fn() {
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
bool fu_make_map(CUtensorMap* map, const void* base, int rows, int K, int box_rows) {
    EncodeTiledFn fn = fu_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)FU_BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t fu_attributes() {
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(gemm_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 112 * 1024);
        // two CTAs of ~100 KB share an SM only if the SM's L1/shared split gives shared memory its maximum
        if (attr_err == cudaSuccess)
            attr_err = cudaFuncSetAttribute(gemm_fused_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    });
    return attr_err;
}

// Cluster size = number of K ranges: the one that keeps the 296 CTA slots (two per SM) busiest over whole rounds of
// tiles, smaller on near ties; every range must keep at least four k-blocks.  (The occupancy calculator is of no help
// here: it reports one CTA per SM for every kernel that allocates tensor memory, whereas two are resident in fact —
// the clock-stamp build counts them.)
struct FuPlan { bool ok; int cluster, clusters, stages, m_pad, n_mma, acc_cols; size_t smem; };
FuPlan fu_plan(int M, int tiles, int K) {
    FuPlan pl{};
    pl.m_pad = (M + 7) / 8 * 8;
    pl.n_mma = 2 * pl.m_pad;
    if (M < 1 || pl.n_mma > 128 || K % FU_BK != 0) return pl;          // two CTAs per SM need 2 x 2 x acc_cols <= 512 columns
    pl.acc_cols = 32;
    while (pl.acc_cols < pl.n_mma) pl.acc_cols *= 2;
    const int kblocks = K / FU_BK;
    const size_t stage = FU_A_BYTES + (size_t)pl.n_mma * FU_BK * 2, staging = (size_t)pl.m_pad * FU_BM * 4;
    pl.stages = (int)std::min<size_t>(FU_MAX_STAGES, (110 * 1024 - staging) / stage);
    if (pl.stages < 3) return pl;
    pl.smem = pl.stages * stage + staging + 1024;
    double best = 0.0;
    for (int c = 2; c <= FU_MAX_CLUSTER && c * 4 <= kblocks; ++c) {
        const int clusters = std::min(FU_CTAS / c, tiles), rounds = (tiles + clusters - 1) / clusters;
        const double balance = (double)tiles * c / ((double)rounds * FU_CTAS);     // busy CTA slots over the kernel's span
        if (balance > best * 1.02) { best = balance; pl.cluster = c; pl.clusters = clusters; }
    }
    pl.ok = pl.cluster >= 2 && best >= 0.8;
    return pl;
}

cudaError_t fu_launch(const void* x, const void* x_lo, const void* w, int w_rows, int box_rows, FuParams& p, const FuPlan& pl,
                      cudaStream_t st) {
    const cudaError_t attr_err = fu_attributes();
    if (attr_err != cudaSuccess) return attr_err;
    CUtensorMap map_w, map_x, map_xlo;
    if (!fu_make_map(&map_w, w, w_rows, p.K, box_rows) || !fu_make_map(&map_x, x, p.M, p.K, p.m_pad) ||
        !fu_make_map(&map_xlo, x_lo, p.M, p.K, p.m_pad))
        return cudaErrorInvalidValue;
    const int clusters = pl.clusters;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(clusters * pl.cluster); cfg.blockDim = dim3(FU_THREADS); cfg.dynamicSmemBytes = pl.smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    attr[n_attr].id = cudaLaunchAttributeClusterDimension;
    attr[n_attr].val.clusterDim.x = pl.cluster; attr[n_attr].val.clusterDim.y = 1; attr[n_attr].val.clusterDim.z = 1;
    ++n_attr;
    if (chain_active()) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    cfg.attrs = attr; cfg.numAttrs = n_attr;
    count_launch();
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemm_fused_kernel, map_w, map_x, map_xlo, p);
    return e != cudaSuccess ? e : cudaGetLastError();
}

void fu_common(FuParams& p, const FuPlan& pl, int mode, int M, int N, int K, int tiles, int* status) {
    p.mode = mode; p.M = M; p.N = N; p.K = K;
    p.m_pad = pl.m_pad; p.n_mma = pl.n_mma; p.acc_cols = pl.acc_cols; p.kblocks = K / FU_BK; p.tiles = tiles;
    p.stages = pl.stages; p.cluster = pl.cluster; p.status = status;
}

bool fu_aligned(const void* a, const void* b, const void* c) { return (((uintptr_t)a | (uintptr_t)b | (uintptr_t)c) % 16) == 0; }

}  // namespace

#ifdef TRJ_TIMELINE
cudaError_t timeline_reset_fused(cudaStream_t st) { return tl::reset(st); }
int timeline_read_fused(int kind, int max_launches, uint64_t* b, uint64_t* e) { return tl::read(kind, max_launches, b, e); }
int timeline_fused_ctas_per_sm() { return tl::sm_peak(); }
#endif

bool gemm_rope_fused_supported(int32_t M, int32_t H, int32_t Hkv, int32_t D, int32_t K, int32_t dtype) {
    return dtype == TRJ_BF16 && D == FU_BM && fu_encode_fn() != nullptr && fu_plan(M, H + 2 * Hkv, K).ok;
}

cudaError_t launch_gemm_rope_fused(const void* x, const void* x_lo, const void* wqkv, int32_t K, const double* inv_freq,
                                   const int32_t* depth, const Batch& bt, void* q_out, void* k_slab, void* v_slab,
                                   int32_t H, int32_t Hkv, int32_t max_seq, int* status, cudaStream_t st) {
    const int tiles = H + 2 * Hkv, M = bt.rows_total;
    const FuPlan pl = fu_plan(M, tiles, K);
    if (!pl.ok || !x_lo || !fu_aligned(x, x_lo, wqkv)) return cudaErrorInvalidValue;
    FuParams p{};
    fu_common(p, pl, FU_ROPE, M, tiles * FU_BM, K, tiles, status);
    p.inv_freq = inv_freq; p.depth = depth; p.seq_len = bt.seq_len; p.row_off = bt.row_off; p.B = bt.B;
    p.H = H; p.Hkv = Hkv; p.max_seq = max_seq;
    p.q_out = (__nv_bfloat16*)q_out; p.k_slab = (__nv_bfloat16*)k_slab; p.v_slab = (__nv_bfloat16*)v_slab;
    return fu_launch(x, x_lo, wqkv, tiles * FU_BM, 64, p, pl, st);
}

bool gemm_swiglu_fused_supported(int32_t M, int32_t f, int32_t K, int32_t dtype) {
    return dtype == TRJ_BF16 && f % 64 == 0 && fu_encode_fn() != nullptr && fu_plan(M, f / 64, K).ok;
}

cudaError_t launch_gemm_swiglu_fused(const void* x, const void* x_lo, const void* w_gate_up, int32_t M, int32_t f, int32_t K,
                                     void* act, void* act_lo, int* status, cudaStream_t st) {
    const int tiles = f / 64;
    const FuPlan pl = fu_plan(M, tiles, K);
    if (!pl.ok || !x_lo || !act_lo || !fu_aligned(x, x_lo, w_gate_up)) return cudaErrorInvalidValue;
    FuParams p{};
    fu_common(p, pl, FU_SWIGLU, M, 2 * f, K, tiles, status);
    p.pair_offset = f; p.f = f;
    p.act = (__nv_bfloat16*)act; p.act_lo = (__nv_bfloat16*)act_lo;
    return fu_launch(x, x_lo, w_gate_up, 2 * f, 64, p, pl, st);
}

}  // namespace trj
