// Shape-generic kernels of the verification step (fp32 or bf16 storage, fp32 arithmetic).
// They serve every shape the specialised sm_100a kernels do not cover (fp32 models, odd head
// sizes) and all the small element-wise steps between the projections.
#include <atomic>
#include <mutex>
#include <algorithm>
#include "trj_internal.h"
#include "timeline.cuh"

namespace trj {
namespace {

// Index checks: a cache row index that a device-held length or path would push outside the cache is never
// dereferenced: the access is skipped (one compare per row; the step's result is then unspecified, since the
// caller's contract seq_len[b] + rows <= max_seq is broken, but no memory outside the cache is touched and nothing
// traps).  The debug build (-DTRJ_DEBUG) also records which check fired in a flag word.
#ifdef TRJ_DEBUG
static __device__ int g_debug_flags;
#define TRJ_DEBUG_CHECK(ok, bit) ((ok) ? true : (atomicOr(&g_debug_flags, (bit)), false))
#else
#define TRJ_DEBUG_CHECK(ok, bit) (ok)
#endif
enum { DBG_ROPE_ROW = 1, DBG_COMPACT_ROW = 2, DBG_ATTENTION_LEN = 4 };

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Activations that feed a projection keep (almost) fp32 precision in bf16 models: the value is
// stored as a bf16 pair hi + lo (lo = the rounding error of hi), which the projection adds back.
template <typename T>
__device__ __forceinline__ void store_split(T* hi, T* lo, size_t i, float v) {
    const T h = from_f<T>(v);
    hi[i] = h;
    if (lo) lo[i] = from_f<T>(v - to_f(h));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Sum of the split-K pieces of a projection result at flat index i (fixed order).
__device__ __forceinline__ float parts_at(const Parts& p, size_t i) {
    float v = p.ptr[i];
    for (int s = 1; s < p.splits; ++s) v += p.ptr[(size_t)s * p.stride + i];
    return v;
}
__device__ __forceinline__ float4 parts_at4(const Parts& p, size_t i4) {
    float4 v = reinterpret_cast<const float4*>(p.ptr)[i4];
    for (int s = 1; s < p.splits; ++s) {
        const float4 b = reinterpret_cast<const float4*>(p.ptr + (size_t)s * p.stride)[i4];
        v.x += b.x; v.y += b.y; v.z += b.z; v.w += b.w;
    }
    return v;
}

// Same for four consecutive values.  The pieces are requested eight at a time before any is added, so the
// loads overlap; the additions keep the order of the pieces.
__device__ __forceinline__ float4 parts_at4_batched(const Parts& p, size_t i4) {
    constexpr int BATCH = 8;
    float4 v = reinterpret_cast<const float4*>(p.ptr)[i4];
    for (int s0 = 1; s0 < p.splits; s0 += BATCH) {
        float4 b[BATCH];
#pragma unroll
        for (int j = 0; j < BATCH; ++j)
            if (s0 + j < p.splits) b[j] = reinterpret_cast<const float4*>(p.ptr + (size_t)(s0 + j) * p.stride)[i4];
#pragma unroll
        for (int j = 0; j < BATCH; ++j)
            if (s0 + j < p.splits) { v.x += b[j].x; v.y += b[j].y; v.z += b[j].z; v.w += b[j].w; }
    }
    return v;
}

// Sequence that owns a global row (B is small: linear scan of the offsets).
__device__ __forceinline__ int seq_of_row(const int32_t* row_off, int B, int row) {
    int b = 0;
    while (b + 1 < B && row >= row_off[b + 1]) ++b;
    return b;
}

// ---------------------------------------------------------------- embedding
template <typename T>
__global__ void embed_kernel(const T* __restrict__ embed, const int32_t* __restrict__ tokens,
                             float* __restrict__ h, int d) {
    pdl_wait();                                  // the chain's fence: everything enqueued earlier is complete
    pdl_launch_dependents();                     // before any later kernel of the chain may start
    TRJ_TL_DECL; TRJ_TL_BEGIN(TRJ_TL_EMBED);
    const int row = blockIdx.x;
    const T* src = embed + (size_t)tokens[row] * d;
    constexpr int VEC = 16 / (int)sizeof(T);                 // elements per 16-byte load
    if (d % VEC == 0 && ((uintptr_t)embed % 16) == 0 && ((uintptr_t)h % 16) == 0) {
        // the table's rows are cold in HBM: few wide loads per thread, all in flight at once
        for (int c = threadIdx.x * VEC; c < d; c += blockDim.x * VEC) {
            const uint4 raw = *reinterpret_cast<const uint4*>(src + c);
            const T* e = reinterpret_cast<const T*>(&raw);
            float out[VEC];
#pragma unroll
            for (int i = 0; i < VEC; ++i) out[i] = to_f(e[i]);
#pragma unroll
            for (int i = 0; i < VEC; i += 4)
                *reinterpret_cast<float4*>(h + (size_t)row * d + c + i) = make_float4(out[i], out[i + 1], out[i + 2], out[i + 3]);
        }
    } else {
        for (int c = threadIdx.x; c < d; c += blockDim.x) h[(size_t)row * d + c] = to_f(src[c]);
    }
    TRJ_TL_END(TRJ_TL_EMBED);
}

// ---------------------------------------------------------------- residual add + RMSNorm
// One CTA per row.  h += add (summing the split-K pieces of `add` on the way), x = rmsnorm(h) * gain.
// Fast path: d % 4 == 0 and d <= 4 * RMS_THREADS * RMS_CHUNKS; the row lives in registers between the two phases.
constexpr int RMS_THREADS = 1024;             // many loads in flight: the row and its split-K pieces come from L2
constexpr int RMS_CHUNKS = 2;

__device__ __forceinline__ float block_sum(float v, float* red) {
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x < 32) {
        float t = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
        t = warp_sum(t);
        if (threadIdx.x == 0) red[0] = t;
    }
    __syncthreads();
    return red[0];
}

template <typename T>
__device__ __forceinline__ void store_split4(T* hi, T* lo, size_t i, float4 v);
template <>
__device__ __forceinline__ void store_split4<float>(float* hi, float*, size_t i, float4 v) {
    *reinterpret_cast<float4*>(hi + i) = v;
}
template <>
__device__ __forceinline__ void store_split4<__nv_bfloat16>(__nv_bfloat16* hi, __nv_bfloat16* lo, size_t i, float4 v) {
    const __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&a); pk.y = *reinterpret_cast<const uint32_t*>(&b);
    *reinterpret_cast<uint2*>(hi + i) = pk;
    if (lo) {
        const __nv_bfloat162 c = __floats2bfloat162_rn(v.x - __low2float(a), v.y - __high2float(a));
        const __nv_bfloat162 e = __floats2bfloat162_rn(v.z - __low2float(b), v.w - __high2float(b));
        pk.x = *reinterpret_cast<const uint32_t*>(&c); pk.y = *reinterpret_cast<const uint32_t*>(&e);
        *reinterpret_cast<uint2*>(lo + i) = pk;
    }
}

template <typename T>
__global__ void __launch_bounds__(RMS_THREADS) add_rmsnorm_vec_kernel(float* __restrict__ h, const Parts add,
                                                                     const float* __restrict__ gain, T* __restrict__ x,
                                                                     T* __restrict__ x_lo, int d, float eps) {
    pdl_prologue();
    TRJ_TL_DECL; TRJ_TL_BEGIN(TRJ_TL_RMSNORM);
    __shared__ float red[32];
    const int row = blockIdx.x, n4 = d >> 2;
    float4 v[RMS_CHUNKS];
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < RMS_CHUNKS; ++k) {
        const int j = threadIdx.x + k * RMS_THREADS;
        if (j < n4) {
            v[k] = reinterpret_cast<const float4*>(h + (size_t)row * d)[j];
            if (add.ptr) {
                // one piece after the other: requesting them together was measured slower inside the step (4.2 against
                // 3.9 us), where the next projection's weight ring is filling at the same time
                const float4 a = parts_at4(add, (size_t)row * n4 + j);
                v[k].x += a.x; v[k].y += a.y; v[k].z += a.z; v[k].w += a.w;
                reinterpret_cast<float4*>(h + (size_t)row * d)[j] = v[k];
            }
            ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
        }
    }
    const float inv = rsqrtf(block_sum(ss, red) / (float)d + eps);
#pragma unroll
    for (int k = 0; k < RMS_CHUNKS; ++k) {
        const int j = threadIdx.x + k * RMS_THREADS;
        if (j < n4) {
            const float4 g = reinterpret_cast<const float4*>(gain)[j];
            store_split4<T>(x, x_lo, (size_t)row * d + 4 * j,
                            make_float4(v[k].x * inv * g.x, v[k].y * inv * g.y, v[k].z * inv * g.z, v[k].w * inv * g.w));
        }
    }
#ifdef TRJ_TIMELINE
    __syncthreads();
#endif
    TRJ_TL_END(TRJ_TL_RMSNORM);
}

template <typename T>
__global__ void add_rmsnorm_kernel(float* __restrict__ h, const Parts add,
                                   const float* __restrict__ gain, T* __restrict__ x, T* __restrict__ x_lo,
                                   int d, float eps) {
    pdl_prologue();
    __shared__ float red[32];
    const int row = blockIdx.x;
    float* hr = h + (size_t)row * d;
    float ss = 0.f;
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
        float v = hr[c];
        if (add.ptr) { v += parts_at(add, (size_t)row * d + c); hr[c] = v; }
        ss += v * v;
    }
    const float inv = rsqrtf(block_sum(ss, red) / (float)d + eps);
    for (int c = threadIdx.x; c < d; c += blockDim.x) store_split(x, x_lo, (size_t)row * d + c, hr[c] * inv * gain[c]);
}

// ---------------------------------------------------------------- plain tiled GEMM
// y[M][N] = (x + x_lo)[M][K] . w[N][K]^T ; 64x64 tile, 16-deep slices, 4x4 outputs per thread.
template <typename T>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T* __restrict__ x, const T* __restrict__ x_lo,
                                                        const T* __restrict__ w, float* __restrict__ y,
                                                        int M, int N, int K) {
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float xs[BK][BM + 4];
    __shared__ float ws[BK][BN + 4];
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int lr = tid >> 2, lk = (tid & 3) * 4;          // this thread stages row lr, k-slice lk..lk+3
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int k = k0 + lk + i;
            const int xm = m0 + lr, wn = n0 + lr;
            float xv = 0.f;
            if (xm < M && k < K) {
                xv = to_f(x[(size_t)xm * K + k]);
                if (x_lo) xv += to_f(x_lo[(size_t)xm * K + k]);
            }
            xs[lk + i][lr] = xv;
            ws[lk + i][lr] = (wn < N && k < K) ? to_f(w[(size_t)wn * K + k]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = xs[kk][ty * 4 + i]; b[i] = ws[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n < N) y[(size_t)m * N + n] = acc[i][j];
        }
    }
}

// ---------------------------------------------------------------- rotary embedding + K/V append
template <typename T>
__global__ void rope_kv_write_kernel(const Parts qkv, const double* __restrict__ inv_freq,
                                     const int32_t* __restrict__ depth, const int32_t* __restrict__ seq_len,
                                     const int32_t* __restrict__ row_off, int B, T* __restrict__ q_out,
                                     T* __restrict__ k_slab, T* __restrict__ v_slab, int H, int Hkv, int D, int max_seq) {
    pdl_launch_dependents();
    // geometry and the rotation of this thread's first element do not depend on the projection: have them
    // ready before waiting for it
    const int row = blockIdx.x, hh = blockIdx.y;
    const int b = seq_of_row(row_off, B, row);
    const int local = row - row_off[b];
    const int pos = seq_len[b] + depth[row];
    const int half = D >> 1, HD = H * D, KD = Hkv * D;
    const bool has_kv = hh < Hkv;                            // this CTA also handles K/V head hh
    const size_t src = (size_t)row * (HD + 2 * KD) + hh * D; // flat index of query head hh in the projection result
    const size_t cache_row = (((size_t)b * Hkv + hh) * max_seq + seq_len[b] + local) * D;
    auto rotation = [&](int i, float& sn, float& cs) {
        // angle in fp64 (positions reach thousands of radians), reduced to [-pi, pi] there; sin/cos of the reduced
        // angle in fp32 are then accurate to ~1e-7
        const double ang = (double)pos * inv_freq[i];
        const double red = ang - 6.283185307179586476925 * rint(ang * 0.15915494309189533577);
        sincosf((float)red, &sn, &cs);
    };
    float sn = 0.f, cs = 1.f;
    if ((int)threadIdx.x < half) rotation(threadIdx.x, sn, cs);
    pdl_wait();
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        if (i != (int)threadIdx.x) rotation(i, sn, cs);
        // all loads first: the stores below could alias them as far as the compiler knows
        float qa = 0.f, qb = 0.f, ka = 0.f, kb = 0.f, va = 0.f, vb = 0.f;
        for (int s = 0; s < qkv.splits; ++s) {               // six independent loads per split-K piece
            const float* piece = qkv.ptr + (size_t)s * qkv.stride + src + i;
            qa += piece[0];      qb += piece[half];
            if (has_kv) {
                ka += piece[HD];      kb += piece[HD + half];
                va += piece[HD + KD]; vb += piece[HD + KD + half];
            }
        }
        q_out[(size_t)row * HD + hh * D + i] = from_f<T>(qa * cs - qb * sn);
        q_out[(size_t)row * HD + hh * D + i + half] = from_f<T>(qb * cs + qa * sn);
        if (!has_kv || !TRJ_DEBUG_CHECK((unsigned)(seq_len[b] + local) < (unsigned)max_seq, DBG_ROPE_ROW)) continue;
        k_slab[cache_row + i] = from_f<T>(ka * cs - kb * sn);
        k_slab[cache_row + i + half] = from_f<T>(kb * cs + ka * sn);
        v_slab[cache_row + i] = from_f<T>(va);
        v_slab[cache_row + i + half] = from_f<T>(vb);
    }
}

// Four consecutive dimensions per thread (head_dim / 2 a multiple of 4): 16-byte loads of the projection pieces,
// 8-byte (bf16) or 16-byte (fp32) stores.  One CTA covers heads_per_cta heads of a row (at most ROPE_THREADS threads).
constexpr int ROPE_THREADS = 256;           // a few fat CTAs (16 heads of 128 each) measured faster than many thin ones
template <typename T>
__global__ void __launch_bounds__(ROPE_THREADS) rope_kv_write_vec_kernel(const Parts qkv, const double* __restrict__ inv_freq,
                                         const int32_t* __restrict__ depth, const int32_t* __restrict__ seq_len,
                                         const int32_t* __restrict__ row_off, int B, T* __restrict__ q_out,
                                         T* __restrict__ k_slab, T* __restrict__ v_slab, int H, int Hkv, int D, int max_seq,
                                         int heads_per_cta) {
    pdl_launch_dependents();
    // geometry and rotations do not depend on the projection: have them ready before waiting for it
    const int half = D >> 1, HD = H * D, KD = Hkv * D, per_head = half >> 2;
    const int row = blockIdx.x, hh = blockIdx.y * heads_per_cta + (int)threadIdx.x / per_head;
    const int i = ((int)threadIdx.x % per_head) * 4;
    TRJ_TL_DECL;
    if (hh >= H) return;                                     // never thread 0: a CTA's first thread has a head
    const int b = seq_of_row(row_off, B, row);
    const int local = row - row_off[b];
    const int pos = seq_len[b] + depth[row];
    const bool has_kv = hh < Hkv;                            // this thread also handles K/V head hh
    const int n_e = has_kv ? 6 : 2;
    const size_t src = (size_t)row * (HD + 2 * KD) + hh * D + i;    // flat index of query head hh in the projection result
    const size_t cache_at = (((size_t)b * Hkv + hh) * max_seq + seq_len[b] + local) * D + i;
    const size_t q_at = (size_t)row * HD + hh * D + i;
    float sn[4], cs[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        // angle in fp64 (positions reach thousands of radians), reduced to [-pi, pi] there; sin/cos of the reduced
        // angle in fp32 are then accurate to ~1e-7
        const double ang = (double)pos * inv_freq[i + e];
        const double red = ang - 6.283185307179586476925 * rint(ang * 0.15915494309189533577);
        sincosf((float)red, &sn[e], &cs[e]);
    }
    pdl_wait();
    TRJ_TL_BEGIN(TRJ_TL_ROPE);
    float4 acc[6];                                           // q, k, v: first and second half of the head
#pragma unroll
    for (int e = 0; e < 6; ++e) acc[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    // the pieces are requested three at a time (18 loads in flight) and added in ascending order
    for (int s0 = 0; s0 < qkv.splits; s0 += 3) {
        float4 t[3][6];
#pragma unroll
        for (int j = 0; j < 3; ++j)
            if (s0 + j < qkv.splits) {
                const float* piece = qkv.ptr + (size_t)(s0 + j) * qkv.stride + src;
#pragma unroll
                for (int e = 0; e < 6; ++e)                  // q at 0, k at HD, v at HD + KD; first and second half of the head
                    if (e < n_e) t[j][e] = *reinterpret_cast<const float4*>(piece + (e >> 1 == 0 ? 0 : e >> 1 == 1 ? HD : HD + KD) + (e & 1) * half);
            }
#pragma unroll
        for (int j = 0; j < 3; ++j)
            if (s0 + j < qkv.splits) {
#pragma unroll
                for (int e = 0; e < 6; ++e)
                    if (e < n_e) { acc[e].x += t[j][e].x; acc[e].y += t[j][e].y; acc[e].z += t[j][e].z; acc[e].w += t[j][e].w; }
            }
    }
    auto rot_lo = [&](const float4& a, const float4& bb) {
        return make_float4(a.x * cs[0] - bb.x * sn[0], a.y * cs[1] - bb.y * sn[1], a.z * cs[2] - bb.z * sn[2], a.w * cs[3] - bb.w * sn[3]);
    };
    auto rot_hi = [&](const float4& a, const float4& bb) {
        return make_float4(bb.x * cs[0] + a.x * sn[0], bb.y * cs[1] + a.y * sn[1], bb.z * cs[2] + a.z * sn[2], bb.w * cs[3] + a.w * sn[3]);
    };
    store_split4<T>(q_out, nullptr, q_at, rot_lo(acc[0], acc[1]));
    store_split4<T>(q_out, nullptr, q_at + half, rot_hi(acc[0], acc[1]));
    if (has_kv && TRJ_DEBUG_CHECK((unsigned)(seq_len[b] + local) < (unsigned)max_seq, DBG_ROPE_ROW)) {
        store_split4<T>(k_slab, nullptr, cache_at, rot_lo(acc[2], acc[3]));
        store_split4<T>(k_slab, nullptr, cache_at + half, rot_hi(acc[2], acc[3]));
        store_split4<T>(v_slab, nullptr, cache_at, acc[4]);
        store_split4<T>(v_slab, nullptr, cache_at + half, acc[5]);
    }
    TRJ_TL_END(TRJ_TL_ROPE);                                 // thread 0's own stores; the others' end within the same few hundred ns
}

// ---------------------------------------------------------------- tree attention, one CTA per (row, head)
// 4 warps split the keys; inside a warp every lane scores one key of a 32-key chunk, the chunk's
// statistics are merged with an online softmax, and P.V is accumulated with lanes spread over D.
template <typename T, int D>
__global__ void __launch_bounds__(128) tree_attention_generic_kernel(
        const T* __restrict__ q, const T* __restrict__ k_slab, const T* __restrict__ v_slab,
        const uint64_t* __restrict__ anc, int anc_words, const int32_t* __restrict__ seq_len,
        const int32_t* __restrict__ row_off, int B, int H, int Hkv, int max_seq, T* __restrict__ out, T* __restrict__ out_lo,
        int shared_cache) {
    constexpr int PER = D / 32;                  // output dims per lane
    __shared__ float qs[D];
    __shared__ float part_m[4], part_l[4];
    __shared__ float part_acc[4][D];
    const int row = blockIdx.x, hh = blockIdx.y;
    const int b = seq_of_row(row_off, B, row);
    const int S = min(max(seq_len[b], 0), max_seq);      // a length outside the cache reads nothing outside it
    const int rows_b = row_off[b + 1] - row_off[b];
    const int total = TRJ_DEBUG_CHECK(seq_len[b] >= 0 && S + rows_b <= max_seq, DBG_ATTENTION_LEN) ? S + rows_b : min(S + rows_b, max_seq);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kvh = hh / (H / Hkv);              // grouped-query attention: the K/V head of this query head
    const int cb = shared_cache ? 0 : b;         // pieces of one prompt chunk share the cache of sequence 0
    const T* kb = k_slab + ((size_t)cb * Hkv + kvh) * max_seq * D;
    const T* vb = v_slab + ((size_t)cb * Hkv + kvh) * max_seq * D;
    const uint64_t* mask = anc + (size_t)row * anc_words;
    for (int c = threadIdx.x; c < D; c += blockDim.x) qs[c] = to_f(q[((size_t)row * H + hh) * D + c]);
    __syncthreads();
    const float scale = rsqrtf((float)D);
    float m_run = -INFINITY, l_run = 0.f, acc[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) acc[i] = 0.f;
    for (int base = warp * 32; base < total; base += 128) {
        const int j = base + lane;
        bool vis = j < total;
        if (vis && j >= S) { const int t = j - S; vis = (mask[t >> 6] >> (t & 63)) & 1ull; }
        float s = -INFINITY;
        if (vis) {
            const T* kr = kb + (size_t)j * D;
            float dot = 0.f;
#pragma unroll 8
            for (int c = 0; c < D; ++c) dot = fmaf(qs[c], to_f(kr[c]), dot);
            s = dot * scale;
        }
        const float cmax = warp_max(s);
        if (cmax == -INFINITY) continue;          // whole chunk masked (warp-uniform)
        const float m_new = fmaxf(m_run, cmax);
        const float corr = (m_run == -INFINITY) ? 0.f : expf(m_run - m_new);
        const float p = vis ? expf(s - m_new) : 0.f;
        l_run = l_run * corr + warp_sum(p);
#pragma unroll
        for (int i = 0; i < PER; ++i) acc[i] *= corr;
        const int nk = min(32, total - base);
        for (int jj = 0; jj < nk; ++jj) {
            const float pj = __shfl_sync(0xffffffffu, p, jj);
            if (pj == 0.f) continue;              // warp-uniform
            const T* vr = vb + (size_t)(base + jj) * D + lane * PER;
#pragma unroll
            for (int i = 0; i < PER; ++i) acc[i] = fmaf(pj, to_f(vr[i]), acc[i]);
        }
        m_run = m_new;
    }
    if (lane == 0) { part_m[warp] = m_run; part_l[warp] = l_run; }
#pragma unroll
    for (int i = 0; i < PER; ++i) part_acc[warp][lane * PER + i] = acc[i];
    __syncthreads();
    const float m_all = fmaxf(fmaxf(part_m[0], part_m[1]), fmaxf(part_m[2], part_m[3]));
    for (int c = threadIdx.x; c < D; c += blockDim.x) {
        float l = 0.f, o = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float f = (part_m[w] == -INFINITY) ? 0.f : expf(part_m[w] - m_all);
            l += part_l[w] * f;
            o += part_acc[w][c] * f;
        }
        store_split(out, out_lo, ((size_t)row * H + hh) * D + c, o / l);
    }
}

// ---------------------------------------------------------------- SwiGLU
template <typename T>
__global__ void swiglu_kernel(const Parts gu, T* __restrict__ act, T* __restrict__ act_lo,
                              int rows, int f) {
    pdl_prologue();
    const size_t n = (size_t)rows * f;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const size_t r = i / f, c = i % f;
        const float g = parts_at(gu, r * 2 * f + c), u = parts_at(gu, r * 2 * f + f + c);
        store_split(act, act_lo, i, g / (1.f + expf(-g)) * u);
    }
}

// Four columns per thread (f a multiple of 4).
template <typename T>
__global__ void swiglu_vec_kernel(const Parts gu, T* __restrict__ act, T* __restrict__ act_lo, int rows, int f) {
    pdl_prologue();
    TRJ_TL_DECL; TRJ_TL_BEGIN(TRJ_TL_SWIGLU);
    const int f4 = f >> 2;
    const size_t n4 = (size_t)rows * f4;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        const size_t r = i / f4, c4 = i % f4;
        const float4 g = parts_at4_batched(gu, r * 2 * f4 + c4), u = parts_at4_batched(gu, r * 2 * f4 + f4 + c4);
        store_split4<T>(act, act_lo, 4 * i,
                        make_float4(g.x / (1.f + expf(-g.x)) * u.x, g.y / (1.f + expf(-g.y)) * u.y,
                                    g.z / (1.f + expf(-g.z)) * u.z, g.w / (1.f + expf(-g.w)) * u.w));
    }
#ifdef TRJ_TIMELINE
    __syncthreads();
#endif
    TRJ_TL_END(TRJ_TL_SWIGLU);
}

// ---------------------------------------------------------------- arg-max + acceptance
// Candidate of a (partial) row scan: best value/index and the runner-up value.
struct Top { float v1; int i1; float v2; };
__device__ __forceinline__ Top top_merge(const Top& a, const Top& b) {
    const bool a_wins = (a.v1 > b.v1) || (a.v1 == b.v1 && a.i1 < b.i1);
    Top r;
    r.v1 = a_wins ? a.v1 : b.v1;
    r.i1 = a_wins ? a.i1 : b.i1;
    r.v2 = fmaxf(a_wins ? b.v1 : a.v1, fmaxf(a.v2, b.v2));
    return r;
}
__device__ __forceinline__ void top_push(Top& t, float v, int i) {
    if (v > t.v1 || (v == t.v1 && i < t.i1)) { t.v2 = fmaxf(t.v2, t.v1); t.v1 = v; t.i1 = i; }
    else t.v2 = fmaxf(t.v2, v);
}
__device__ __forceinline__ Top top_shfl_xor(const Top& t, int o) {
    Top r;
    r.v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
    r.i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
    r.v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
    return r;
}

constexpr int ARGMAX_THREADS = 256;
constexpr int ARGMAX_CHUNKS = 8;              // vocabulary slices per row (one CTA each)

// The acceptance walk of one sequence, run by one CTA after every prediction of it is known.
__device__ void accept_sequence(const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                const int32_t* pred, int rows, int32_t* k_acc, int32_t* path, int32_t* bonus) {
    rows = min(rows, TRJ_MAX_ROWS);              // the host refuses larger trees; a bad device-side row_off must not overrun
    __shared__ unsigned char ok[TRJ_MAX_ROWS];
    __shared__ int32_t s_tok[TRJ_MAX_ROWS], s_par[TRJ_MAX_ROWS], s_dep[TRJ_MAX_ROWS], s_pred[TRJ_MAX_ROWS];
    __shared__ int s_best;
    // all threads fetch the tree, then one thread walks it out of shared memory
    for (int i = threadIdx.x; i < rows; i += blockDim.x) {
        s_tok[i] = tokens[i]; s_par[i] = parent[i]; s_dep[i] = depth[i];
        s_pred[i] = __ldcg(pred + i);            // possibly written by other CTAs of this launch: read it from L2
    }
    __syncthreads();
    // ok[i] = every row on the path root..i carries the token its parent predicted.  Pointer jumping: after round r a
    // row has folded in the matches of its 2^r nearest ancestors, so ceil(log2(rows)) rounds replace a serial walk
    // over the rows (the walk was the longest single piece of this kernel).
    __shared__ short jump[2][TRJ_MAX_ROWS];
    __shared__ unsigned char okb[2][TRJ_MAX_ROWS];
    for (int i = threadIdx.x; i < rows; i += blockDim.x) {
        const int p = s_par[i];
        okb[0][i] = i == 0 || s_tok[i] == s_pred[p];
        jump[0][i] = (short)(i == 0 ? 0 : p);
    }
    __syncthreads();
    int cur = 0;
    for (int span = 1; span < rows; span <<= 1, cur ^= 1) {
        for (int i = threadIdx.x; i < rows; i += blockDim.x) {
            const int j = jump[cur][i];
            okb[cur ^ 1][i] = okb[cur][i] && okb[cur][j];
            jump[cur ^ 1][i] = jump[cur][j];
        }
        __syncthreads();
    }
    for (int i = threadIdx.x; i < rows; i += blockDim.x) ok[i] = okb[cur][i];
    __syncthreads();
    if (threadIdx.x == 0) {
        int best = 0, best_depth = 0;
        for (int i = 1; i < rows; ++i)
            if (ok[i] && s_dep[i] > best_depth) { best = i; best_depth = s_dep[i]; }
        *k_acc = best_depth;
        *bonus = s_pred[best];
        int node = best;
        for (int j = best_depth; j >= 0; --j) { path[j] = node; node = s_par[node]; }
        s_best = best_depth;
    }
    __syncthreads();
    for (int j = s_best + 1 + (int)threadIdx.x; j < TRJ_PATH_STRIDE; j += blockDim.x) path[j] = -1;
}

template <typename T>
__global__ void __launch_bounds__(ARGMAX_THREADS) argmax_accept_kernel(
        const T* __restrict__ logits, int V, const int32_t* __restrict__ tokens,
        const int32_t* __restrict__ parent, const int32_t* __restrict__ depth,
        const int32_t* __restrict__ row_off, int B, int32_t* node_argmax,
        float* __restrict__ margin, int32_t* __restrict__ k_acc, int32_t* __restrict__ path,
        int32_t* __restrict__ bonus, int do_accept, unsigned int* tickets, Top* partial) {
    pdl_prologue();
    __shared__ Top red[ARGMAX_THREADS / 32];
    __shared__ int last_flag;
    const int row = blockIdx.x, chunk = blockIdx.y;
    const int per = (V + ARGMAX_CHUNKS - 1) / ARGMAX_CHUNKS;
    const int v0 = chunk * per, v1 = min(V, v0 + per);
    const T* lr = logits + (size_t)row * V;
    Top t{-INFINITY, 0x7fffffff, -INFINITY};
    constexpr int VEC = 16 / (int)sizeof(T);                 // elements per 16-byte load
    if (V % VEC == 0 && per % VEC == 0 && ((uintptr_t)logits % 16) == 0) {
        for (int v = v0 + threadIdx.x * VEC; v < v1; v += ARGMAX_THREADS * VEC) {
            const uint4 raw = *reinterpret_cast<const uint4*>(lr + v);
            const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
            for (int i = 0; i < VEC; ++i) top_push(t, to_f(e[i]), v + i);
        }
    } else {
        for (int v = v0 + threadIdx.x; v < v1; v += ARGMAX_THREADS) top_push(t, to_f(lr[v]), v);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t = top_merge(t, top_shfl_xor(t, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
        Top r = red[0];
        for (int w = 1; w < ARGMAX_THREADS / 32; ++w) r = top_merge(r, red[w]);
        partial[(size_t)row * ARGMAX_CHUNKS + chunk] = r;
        __threadfence();
        const int b = seq_of_row(row_off, B, row);
        const unsigned int need = (unsigned int)(row_off[b + 1] - row_off[b]) * ARGMAX_CHUNKS;
        const unsigned int got = atomicAdd(&tickets[b], 1u);
        last_flag = (got + 1 == need) ? b : -1;
    }
    __syncthreads();
    const int b = last_flag;
    if (b < 0) return;
    // this CTA saw the last slice of sequence b: finish its rows, then walk the tree
    __threadfence();
    const int r0 = row_off[b], rows = row_off[b + 1] - r0;
    for (int i = threadIdx.x; i < rows; i += ARGMAX_THREADS) {
        const volatile Top* pp = partial + (size_t)(r0 + i) * ARGMAX_CHUNKS;
        Top r{pp[0].v1, pp[0].i1, pp[0].v2};
        for (int c = 1; c < ARGMAX_CHUNKS; ++c) { Top o{pp[c].v1, pp[c].i1, pp[c].v2}; r = top_merge(r, o); }
        node_argmax[r0 + i] = r.i1;
        if (margin) margin[r0 + i] = r.v1 - r.v2;
    }
    if (threadIdx.x == 0) tickets[b] = 0;       // ready for the next call
    __syncthreads();
    if (do_accept)
        accept_sequence(tokens + r0, parent + r0, depth + r0, node_argmax + r0, rows,
                        k_acc + b, path + (size_t)b * TRJ_PATH_STRIDE, bonus + b);
}

// ---------------------------------------------------------------- per-row top-K (K = 1: arg-max) + acceptance
// One CTA per row.  Every thread keeps the KMAX best of its share of the row as a sorted list in registers (order:
// larger value first, equal values by ascending id); each warp then merges its 32 lists into one by KMAX rounds of a
// warp-wide arg-max over the lists' heads, and the first warp merges the 32 warp lists the same way.  The CTA that
// finishes the last row of a sequence walks that sequence's tree.
constexpr int TOPK_THREADS = 1024;
// Top-K (K <= TRJ_MAX_TOPK) of a row, value first and the smaller id among equals.  The row is taken in chunks of
// 32 x 1024 elements that the CTA's threads hold in registers (element j * 1024 + t of the chunk in thread t).
// Per chunk: (A) the 32 warp maxima; their K-th largest is a value that at least K elements of the chunk reach, so
// together with the K-th value of the row's running list it is a threshold below which nothing can enter the list;
// (B) every element at or above the threshold goes to a candidate buffer in shared memory (slots handed out by an
// atomic counter: the order in the buffer is arbitrary, the selection below is not); (C) the first warp selects the K
// best among the candidates and the running list by K rounds of a scan and a shuffle reduction.  Typically a few
// dozen elements survive the threshold.  If more survive than the buffer holds (many equal values), the chunk is
// done the slow way: K rounds of selection over all its elements, in every warp and then over the warps' lists.
constexpr int TOPK_PER_THREAD = 32;
constexpr int TOPK_CAND = 1024;
__device__ __forceinline__ bool top_better(float v, int i, float w, int j) { return v > w || (v == w && i < j); }
__device__ __forceinline__ void warp_best(float& bv, int& bi) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (top_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
}
template <typename T>
__global__ void __launch_bounds__(TOPK_THREADS) topk_accept_kernel(
        const T* __restrict__ logits, int V, int K, const int32_t* __restrict__ tokens,
        const int32_t* __restrict__ parent, const int32_t* __restrict__ depth,
        const int32_t* __restrict__ row_off, int B, int32_t* __restrict__ topk, int32_t* node_argmax,
        float* __restrict__ margin, int32_t* __restrict__ k_acc, int32_t* __restrict__ path,
        int32_t* __restrict__ bonus, int do_accept, unsigned int* tickets) {
    pdl_prologue();
    __shared__ float cand_v[TOPK_CAND + TRJ_MAX_TOPK];             // candidates of the chunk, then the running list
    __shared__ int cand_i[TOPK_CAND + TRJ_MAX_TOPK];
    __shared__ float list_v[TOPK_THREADS / 32][TRJ_MAX_TOPK];      // slow path: the warps' sorted lists; [0] also: warp maxima
    __shared__ int list_i[TOPK_THREADS / 32][TRJ_MAX_TOPK];
    __shared__ float best_v[TRJ_MAX_TOPK];                          // the row's running list, sorted
    __shared__ int best_i[TRJ_MAX_TOPK];
    __shared__ float warp_max_v[TOPK_THREADS / 32];
    __shared__ float thr;
    __shared__ int cand_n;
    __shared__ int last_flag;
    const int row = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const T* lr = logits + (size_t)row * V;
    if (tid < TRJ_MAX_TOPK) { best_v[tid] = -INFINITY; best_i[tid] = 0x7fffffff; }
    for (int base = 0; base < V; base += TOPK_PER_THREAD * TOPK_THREADS) {
        float x[TOPK_PER_THREAD];
        float tm = -INFINITY;
#pragma unroll
        for (int j = 0; j < TOPK_PER_THREAD; ++j) {
            const int id = base + j * TOPK_THREADS + tid;
            x[j] = id < V ? to_f(lr[id]) : -INFINITY;
            tm = fmaxf(tm, x[j]);
        }
        // (A) warp maxima, then the K-th largest of them (with multiplicity) in the first warp
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, o));
        if (lane == 0) warp_max_v[warp] = tm;
        __syncthreads();
        if (warp == 0) {
            float mine = warp_max_v[lane], kth = -INFINITY;
            for (int r = 0; r < K; ++r) {
                float m = mine;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                kth = m;
                const unsigned holders = __ballot_sync(0xffffffffu, mine == m);
                if (lane == __ffs(holders) - 1) mine = -INFINITY;      // one holder gives its value up per round
            }
            if (lane == 0) { thr = fmaxf(kth, best_v[K - 1]); cand_n = 0; }
        }
        __syncthreads();
        // (B) candidates
        const float t = thr;
#pragma unroll
        for (int j = 0; j < TOPK_PER_THREAD; ++j) {
            const int id = base + j * TOPK_THREADS + tid;
            if (id < V && x[j] >= t) {
                const int slot = atomicAdd(&cand_n, 1);
                if (slot < TOPK_CAND) { cand_v[slot] = x[j]; cand_i[slot] = id; }
            }
        }
        __syncthreads();
        const int n_cand = cand_n;                           // the same for every thread
        if (n_cand <= TOPK_CAND) {
            // (C) the first warp: K best of the candidates and the running list
            if (warp == 0) {
                if (lane < K) { cand_v[n_cand + lane] = best_v[lane]; cand_i[n_cand + lane] = best_i[lane]; }
                __syncwarp();
                const int n = n_cand + K;
                float mv = -INFINITY;
                int mi = 0x7fffffff;
                for (int r = 0; r < K; ++r) {
                    float bv = -INFINITY;
                    int bi = 0x7fffffff, bs = -1;
                    for (int e = lane; e < n; e += 32) {
                        const float v = cand_v[e];
                        const int i = cand_i[e];
                        if (i != 0x7fffffff && top_better(v, i, bv, bi)) { bv = v; bi = i; bs = e; }
                    }
                    const int mine_i = bi;
                    warp_best(bv, bi);
                    if (bs >= 0 && mine_i == bi) cand_i[bs] = 0x7fffffff;     // taken (ids are unique: one lane owns it)
                    __syncwarp();
                    if (lane == r) { mv = bv; mi = bi; }
                }
                if (lane < K) { best_v[lane] = mv; best_i[lane] = mi; }
            }
        } else {
            // slow path: K rounds over all elements of the chunk in every warp, then over the warps' lists
            uint32_t taken = 0;
            for (int r = 0; r < K; ++r) {
                float bv = -INFINITY;
                int bj = -1;
#pragma unroll
                for (int j = 0; j < TOPK_PER_THREAD; ++j)    // ascending ids: "strictly larger" keeps the smallest id among equals
                    if (!((taken >> j) & 1u) && x[j] > bv) { bv = x[j]; bj = j; }
                int bi = bj >= 0 ? base + bj * TOPK_THREADS + tid : 0x7fffffff;
                const int mine_i = bi;
                warp_best(bv, bi);
                if (bi == mine_i && bj >= 0) taken |= 1u << bj;
                if (lane == 0) { list_v[warp][r] = bv; list_i[warp][r] = bi; }
            }
            __syncthreads();
            if (warp == 0) {
                int head = 0;
                float mv = -INFINITY;
                int mi = 0x7fffffff;
                for (int r = 0; r < K; ++r) {
                    float bv = head < K ? list_v[lane][head] : -INFINITY;
                    int bi = head < K ? list_i[lane][head] : 0x7fffffff;
                    const int mine_i = bi;
                    warp_best(bv, bi);
                    if (bi == mine_i && bi != 0x7fffffff) ++head;
                    if (lane == r) { mv = bv; mi = bi; }
                }
                if (lane < K) { list_v[0][lane] = mv; list_i[0][lane] = mi; }
                __syncwarp();
                if (lane == 0) {                             // two sorted lists of K entries -> the K best
                    float nv[TRJ_MAX_TOPK];
                    int ni[TRJ_MAX_TOPK];
                    int a = 0, c = 0;
                    for (int r = 0; r < K; ++r) {
                        if (top_better(list_v[0][a], list_i[0][a], best_v[c], best_i[c])) { nv[r] = list_v[0][a]; ni[r] = list_i[0][a]; ++a; }
                        else { nv[r] = best_v[c]; ni[r] = best_i[c]; ++c; }
                    }
                    for (int r = 0; r < K; ++r) { best_v[r] = nv[r]; best_i[r] = ni[r]; }
                }
            }
        }
        __syncthreads();                                     // the buffers are rewritten by the next chunk
    }
    if (tid < K && topk) topk[(size_t)row * K + tid] = best_i[tid];
    if (tid == 0) {
        node_argmax[row] = best_i[0];
        if (margin) margin[row] = best_v[0] - best_v[K > 1 ? 1 : 0];
        __threadfence();
        const int b = seq_of_row(row_off, B, row);
        const unsigned int need = (unsigned int)(row_off[b + 1] - row_off[b]);
        const unsigned int got = atomicAdd(&tickets[b], 1u);
        last_flag = (got + 1 == need) ? b : -1;
        if (got + 1 == need) tickets[b] = 0;                 // ready for the next call
    }
    __syncthreads();
    const int b = last_flag;
    if (b < 0 || !do_accept) return;
    __threadfence();                                         // the other rows' predictions were written by other CTAs
    const int r0 = row_off[b], rows = row_off[b + 1] - r0;
    accept_sequence(tokens + r0, parent + r0, depth + r0, node_argmax + r0, rows,
                    k_acc + b, path + (size_t)b * TRJ_PATH_STRIDE, bonus + b);
}

// The arg-max of every verification step (K = 1): one CTA per row, five instructions per element.  A thread scans its
// elements in ascending id order, so "strictly larger" keeps the smallest id among equals; the runner-up value (for
// the margin) is max(v2, min(v1, x)).  Threads, then warps, are merged with the full (value, id) order.
template <typename T>
__global__ void __launch_bounds__(TOPK_THREADS) argmax_row_accept_kernel(
        const T* __restrict__ logits, int V, const int32_t* __restrict__ tokens,
        const int32_t* __restrict__ parent, const int32_t* __restrict__ depth,
        const int32_t* __restrict__ row_off, int B, int32_t* node_argmax,
        float* __restrict__ margin, int32_t* __restrict__ k_acc, int32_t* __restrict__ path,
        int32_t* __restrict__ bonus, int do_accept, unsigned int* tickets) {
    pdl_prologue();
    __shared__ Top red[TOPK_THREADS / 32];
    __shared__ int last_flag;
    const int row = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const T* lr = logits + (size_t)row * V;
    float v1 = -INFINITY, v2 = -INFINITY;
    int i1 = 0x7fffffff;
    auto look = [&](float x, int i) {
        v2 = fmaxf(v2, fminf(v1, x));
        i1 = x > v1 ? i : i1;
        v1 = fmaxf(v1, x);
    };
    constexpr int VEC = 16 / (int)sizeof(T);
    if (V % VEC == 0 && ((uintptr_t)logits % 16) == 0) {
        constexpr int BATCH = 4;                             // four 16-byte loads in flight per thread
        for (int v0 = threadIdx.x * VEC; v0 < V; v0 += BATCH * TOPK_THREADS * VEC) {
            uint4 raw[BATCH];
#pragma unroll
            for (int j = 0; j < BATCH; ++j) {
                const int v = v0 + j * TOPK_THREADS * VEC;
                if (v < V) raw[j] = *reinterpret_cast<const uint4*>(lr + v);
            }
#pragma unroll
            for (int j = 0; j < BATCH; ++j) {
                const int v = v0 + j * TOPK_THREADS * VEC;
                if (v < V) {
                    const T* e = reinterpret_cast<const T*>(&raw[j]);
#pragma unroll
                    for (int i = 0; i < VEC; ++i) look(to_f(e[i]), v + i);
                }
            }
        }
    } else {
        for (int v = threadIdx.x; v < V; v += TOPK_THREADS) look(to_f(lr[v]), v);
    }
    Top t{v1, i1, v2};
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t = top_merge(t, top_shfl_xor(t, o));
    if (lane == 0) red[warp] = t;
    __syncthreads();
    if (warp == 0) {
        t = red[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t = top_merge(t, top_shfl_xor(t, o));
        if (lane == 0) {
            node_argmax[row] = t.i1;
            if (margin) margin[row] = t.v1 - t.v2;
            __threadfence();
            const int b = seq_of_row(row_off, B, row);
            const unsigned int need = (unsigned int)(row_off[b + 1] - row_off[b]);
            const unsigned int got = atomicAdd(&tickets[b], 1u);
            last_flag = (got + 1 == need) ? b : -1;
            if (got + 1 == need) tickets[b] = 0;             // ready for the next call
        }
    }
    __syncthreads();
    const int b = last_flag;
    if (b < 0 || !do_accept) return;
    __threadfence();                                         // the other rows' predictions were written by other CTAs
    const int r0 = row_off[b], rows = row_off[b + 1] - r0;
    accept_sequence(tokens + r0, parent + r0, depth + r0, node_argmax + r0, rows,
                    k_acc + b, path + (size_t)b * TRJ_PATH_STRIDE, bonus + b);
}

// Arg-max of every row from the candidates a projection's epilogue left (one per 32 outputs), then acceptance as above.
__global__ void __launch_bounds__(128) argmax_table_accept_kernel(
        const TopEntry* __restrict__ table, int per_row, const int32_t* __restrict__ tokens,
        const int32_t* __restrict__ parent, const int32_t* __restrict__ depth,
        const int32_t* __restrict__ row_off, int B, int32_t* node_argmax,
        float* __restrict__ margin, int32_t* __restrict__ k_acc, int32_t* __restrict__ path,
        int32_t* __restrict__ bonus, int do_accept, unsigned int* tickets) {
    pdl_prologue();
    __shared__ Top red[4];
    __shared__ int last_flag;
    const int row = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const TopEntry* tr = table + (size_t)row * per_row;
    Top t{-INFINITY, 0x7fffffff, -INFINITY};
    for (int i = threadIdx.x; i < per_row; i += 128) {
        const TopEntry e = tr[i];
        t = top_merge(t, Top{e.v1, e.i1, e.v2});
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t = top_merge(t, top_shfl_xor(t, o));
    if (lane == 0) red[warp] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
        t = top_merge(top_merge(red[0], red[1]), top_merge(red[2], red[3]));
        node_argmax[row] = t.i1;
        if (margin) margin[row] = t.v1 - t.v2;
        __threadfence();
        const int b = seq_of_row(row_off, B, row);
        const unsigned int need = (unsigned int)(row_off[b + 1] - row_off[b]);
        const unsigned int got = atomicAdd(&tickets[b], 1u);
        last_flag = (got + 1 == need) ? b : -1;
        if (got + 1 == need) tickets[b] = 0;                 // ready for the next call
    }
    __syncthreads();
    const int b = last_flag;
    if (b < 0 || !do_accept) return;
    __threadfence();                                         // the other rows' predictions were written by other CTAs
    const int r0 = row_off[b], rows = row_off[b + 1] - r0;
    accept_sequence(tokens + r0, parent + r0, depth + r0, node_argmax + r0, rows,
                    k_acc + b, path + (size_t)b * TRJ_PATH_STRIDE, bonus + b);
}

__global__ void accept_only_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                                   const int32_t* __restrict__ depth, const int32_t* __restrict__ row_off,
                                   const int32_t* __restrict__ node_argmax, int32_t* __restrict__ k_acc,
                                   int32_t* __restrict__ path, int32_t* __restrict__ bonus) {
    pdl_prologue();
    const int b = blockIdx.x, r0 = row_off[b], rows = row_off[b + 1] - r0;
    accept_sequence(tokens + r0, parent + r0, depth + r0, node_argmax + r0, rows,
                    k_acc + b, path + (size_t)b * TRJ_PATH_STRIDE, bonus + b);
}

// ---------------------------------------------------------------- KV compaction
// One CTA per (layer, sequence, head, K|V).  Rows are moved in ascending order in batches that are
// fully loaded before they are stored; since path[j] >= j and the path is strictly increasing, a
// destination never overwrites a row that a later batch still has to read.
constexpr int COMPACT_BATCH = 16;
__global__ void __launch_bounds__(256) compact_kernel(uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                                                      int B_cache, int B, int H, int max_seq, int row_vec,
                                                      int32_t* seq_len,
                                                      const int32_t* __restrict__ k_acc,
                                                      const int32_t* __restrict__ path, unsigned int* tickets) {
    pdl_prologue();
    extern __shared__ uint4 stage[];             // [COMPACT_BATCH][row_vec]
    int idx = blockIdx.x;
    const int kv = idx & 1; idx >>= 1;
    const int hh = idx % H; idx /= H;
    const int b = idx % B; const int l = idx / B;
    const int k = min(k_acc[b], TRJ_PATH_STRIDE - 1);    // a path holds at most TRJ_PATH_STRIDE rows
    const int S = seq_len[b];
    // With tickets the sequence's length is advanced here as well: every CTA has read it by the time it draws its
    // ticket, so the CTA that draws the last one may write it (and leaves the ticket at zero for the next call).
    auto finish = [&]() {
        if (!tickets) return;
        __syncthreads();
        if (threadIdx.x == 0) {
            const unsigned int per_seq = gridDim.x / (unsigned int)B;
            if (atomicAdd(&tickets[b], 1u) + 1u == per_seq) { tickets[b] = 0; seq_len[b] = S + k + 1; }
        }
    };
    if (k <= 0) { finish(); return; }
    uint4* slab = (kv ? v_cache : k_cache) + (((size_t)l * B_cache + b) * H + hh) * (size_t)max_seq * row_vec;
    const int32_t* pb = path + (size_t)b * TRJ_PATH_STRIDE;
    for (int j0 = 1; j0 <= k; j0 += COMPACT_BATCH) {
        const int nj = min(COMPACT_BATCH, k - j0 + 1);
        for (int e = threadIdx.x; e < nj * row_vec; e += blockDim.x) {
            const int j = j0 + e / row_vec, c = e % row_vec;
            if (TRJ_DEBUG_CHECK(pb[j] >= 0 && (unsigned)(S + pb[j]) < (unsigned)max_seq, DBG_COMPACT_ROW))
                stage[e] = slab[(size_t)(S + pb[j]) * row_vec + c];
        }
        __syncthreads();
        for (int e = threadIdx.x; e < nj * row_vec; e += blockDim.x) {
            const int j = j0 + e / row_vec, c = e % row_vec;
            if (TRJ_DEBUG_CHECK(pb[j] >= 0 && (unsigned)(S + pb[j]) < (unsigned)max_seq && (unsigned)(S + j) < (unsigned)max_seq, DBG_COMPACT_ROW))
                slab[(size_t)(S + j) * row_vec + c] = stage[e];
        }
        __syncthreads();
    }
    finish();
}

__global__ void advance_len_kernel(int32_t* seq_len, const int32_t* k_acc, int B) {
    pdl_prologue();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) seq_len[b] += k_acc[b] + 1;
}
__global__ void set_chunk_kernel(int32_t* row_off2, int m) { row_off2[0] = 0; row_off2[1] = m; }
__global__ void prefill_geometry_kernel(const int32_t* seq_len_b, int32_t* lens, int n_sub, int sub, int m, int32_t* off_all,
                                        int32_t* off_pieces) {
    for (int j = threadIdx.x; j < n_sub; j += blockDim.x) lens[j] = *seq_len_b + j * sub;
    for (int j = threadIdx.x; j <= n_sub; j += blockDim.x) off_pieces[j] = min(j * sub, m);
    if (threadIdx.x == 0) { off_all[0] = 0; off_all[1] = m; }
}
__global__ void bump_len_kernel(int32_t* seq_len_b, int delta) { *seq_len_b += delta; }

}  // namespace

// ============================================================================ launchers
static std::atomic<bool> g_pdl{true};
bool pdl_enabled() { return g_pdl.load(std::memory_order_relaxed); }
void set_pdl(bool on) { g_pdl.store(on, std::memory_order_relaxed); }
static thread_local int t_chain_depth = 0;
bool chain_active() { return t_chain_depth > 0 && pdl_enabled(); }
ChainScope::ChainScope() { ++t_chain_depth; }
ChainScope::~ChainScope() { --t_chain_depth; }
#ifdef TRJ_DEBUG
cudaError_t debug_flags_read(int* flags) {
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpyFromSymbol(flags, g_debug_flags, sizeof(int));
    const int zero = 0;
    if (e == cudaSuccess) e = cudaMemcpyToSymbol(g_debug_flags, &zero, sizeof(int));
    return e;
}
#endif
#ifdef TRJ_TIMELINE
cudaError_t timeline_reset_generic(cudaStream_t st) { return tl::reset(st); }
int timeline_read_generic(int kind, int max_launches, uint64_t* b, uint64_t* e) { return tl::read(kind, max_launches, b, e); }
#endif
static std::atomic<uint64_t> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
uint64_t launches_so_far() { return g_launches.load(std::memory_order_relaxed); }

#define DISPATCH_T(dtype, ...)                                         \
    if ((dtype) == TRJ_BF16) { using T = __nv_bfloat16; __VA_ARGS__; } \
    else { using T = float; __VA_ARGS__; }

cudaError_t launch_embed(const void* embed, int32_t dtype, const int32_t* tokens, float* h,
                         int32_t rows, int32_t d, cudaStream_t st) {
    count_launch();
    cudaError_t launch_err = cudaSuccess;
    DISPATCH_T(dtype, launch_err = launch_chain(embed_kernel<T>, dim3(rows), dim3(256), 0, st, (const T*)embed, tokens, h, d));
    return launch_err != cudaSuccess ? launch_err : cudaGetLastError();
}

cudaError_t launch_add_rmsnorm(float* h, const Parts& add, const float* gain, void* x, void* x_lo, int32_t dtype,
                               int32_t rows, int32_t d, float eps, cudaStream_t st) {
    count_launch();
    cudaError_t launch_err = cudaSuccess;
    const bool vec = d % 4 == 0 && d <= 4 * RMS_THREADS * RMS_CHUNKS && add.stride % 4 == 0 &&
                     ((uintptr_t)h | (uintptr_t)add.ptr | (uintptr_t)gain | (uintptr_t)x | (uintptr_t)x_lo) % 16 == 0;
    if (vec) {
        DISPATCH_T(dtype, launch_err = launch_chain(add_rmsnorm_vec_kernel<T>, dim3(rows), dim3(RMS_THREADS), 0, st, h, add, gain, (T*)x, (T*)x_lo, d, eps));
    } else {
        DISPATCH_T(dtype, launch_err = launch_chain(add_rmsnorm_kernel<T>, dim3(rows), dim3(256), 0, st, h, add, gain, (T*)x, (T*)x_lo, d, eps));
    }
    return launch_err != cudaSuccess ? launch_err : cudaGetLastError();
}

cudaError_t launch_gemm_simt(const void* x, const void* x_lo, const void* w, float* y, int32_t M, int32_t N,
                             int32_t K, int32_t dtype, cudaStream_t st) {
    count_launch();
    dim3 grid((N + 63) / 64, (M + 63) / 64);
    DISPATCH_T(dtype, gemm_simt_kernel<T><<<grid, 256, 0, st>>>((const T*)x, (const T*)x_lo, (const T*)w, y, M, N, K));
    return cudaGetLastError();
}

cudaError_t launch_rope_kv_write(const Parts& qkv, const double* inv_freq, const int32_t* depth,
                                 const Batch& bt, void* q_out, void* k_slab, void* v_slab, int32_t dtype,
                                 int32_t H, int32_t Hkv, int32_t D, int32_t max_seq, cudaStream_t st) {
    count_launch();
    cudaError_t launch_err = cudaSuccess;
    const int per_head = D / 8;                              // threads per head in the vector kernel
    const int hpc = per_head > 0 ? std::max(1, std::min(H, ROPE_THREADS / per_head)) : 1;
    const bool vec = D % 8 == 0 && per_head <= ROPE_THREADS && qkv.stride % 4 == 0 && ((uintptr_t)qkv.ptr % 16) == 0;
    if (vec) {
        dim3 grid(bt.rows_total, (H + hpc - 1) / hpc);
        DISPATCH_T(dtype, launch_err = launch_chain(rope_kv_write_vec_kernel<T>, grid, dim3(per_head * hpc), 0, st, qkv, inv_freq, depth,
                                                    bt.seq_len, bt.row_off, bt.B, (T*)q_out, (T*)k_slab, (T*)v_slab, H, Hkv, D, max_seq, hpc));
    } else {
        dim3 grid(bt.rows_total, H);
        DISPATCH_T(dtype, launch_err = launch_chain(rope_kv_write_kernel<T>, grid, dim3(64), 0, st, qkv, inv_freq, depth, bt.seq_len, bt.row_off,
                                                    bt.B, (T*)q_out, (T*)k_slab, (T*)v_slab, H, Hkv, D, max_seq));
    }
    return launch_err != cudaSuccess ? launch_err : cudaGetLastError();
}

cudaError_t launch_tree_attention_generic(const void* q, const void* k_slab, const void* v_slab,
                                          const uint64_t* anc, int32_t anc_words, const Batch& bt,
                                          int32_t H, int32_t Hkv, int32_t D, int32_t max_seq, int32_t dtype,
                                          void* out, void* out_lo, cudaStream_t st) {
    count_launch();
    dim3 grid(bt.rows_total, H);
#define ATT(DD)                                                                                          \
    DISPATCH_T(dtype, tree_attention_generic_kernel<T, DD><<<grid, 128, 0, st>>>(                        \
                          (const T*)q, (const T*)k_slab, (const T*)v_slab, anc, anc_words, bt.seq_len,   \
                          bt.row_off, bt.B, H, Hkv, max_seq, (T*)out, (T*)out_lo, bt.shared_cache))
    if (D == 64) { ATT(64); }
    else if (D == 128) { ATT(128); }
    else return cudaErrorInvalidValue;
#undef ATT
    return cudaGetLastError();
}

cudaError_t launch_swiglu(const Parts& gu, void* act, void* act_lo, int32_t dtype, int32_t rows, int32_t f,
                          cudaStream_t st) {
    count_launch();
    cudaError_t launch_err = cudaSuccess;
    const bool vec = f % 4 == 0 && gu.stride % 4 == 0 && ((uintptr_t)gu.ptr % 16) == 0;
    const size_t n = (size_t)rows * (vec ? f / 4 : f);
    const int blocks = (int)((n + 127) / 128 < 2368 ? (n + 127) / 128 : 2368);
    if (vec) {
        DISPATCH_T(dtype, launch_err = launch_chain(swiglu_vec_kernel<T>, dim3(blocks), dim3(128), 0, st, gu, (T*)act, (T*)act_lo, rows, f));
    } else {
        DISPATCH_T(dtype, launch_err = launch_chain(swiglu_kernel<T>, dim3(blocks), dim3(128), 0, st, gu, (T*)act, (T*)act_lo, rows, f));
    }
    return launch_err != cudaSuccess ? launch_err : cudaGetLastError();
}

size_t argmax_workspace_bytes(int32_t rows_total, int32_t B) {
    (void)B;
    return align_up(sizeof(unsigned int) * TRJ_MAX_BATCH, 256) + align_up(sizeof(Top) * ARGMAX_CHUNKS * (size_t)rows_total, 256);
}

cudaError_t launch_argmax_accept(const void* logits, int32_t dtype, int32_t V,
                                 const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                 const int32_t* row_off, int32_t B, int32_t rows_total,
                                 int32_t* node_argmax, float* margin, int32_t* k_acc, int32_t* path,
                                 int32_t* bonus, bool do_argmax, bool do_accept, void* ws, cudaStream_t st) {
    if (do_argmax || do_accept) count_launch();
    cudaError_t launch_err = cudaSuccess;
    if (do_argmax) {
        unsigned int* tickets = (unsigned int*)ws;
        Top* partial = (Top*)((char*)ws + align_up(sizeof(unsigned int) * TRJ_MAX_BATCH, 256));
        dim3 grid(rows_total, ARGMAX_CHUNKS);
        DISPATCH_T(dtype, launch_err = launch_chain(argmax_accept_kernel<T>, grid, dim3(ARGMAX_THREADS), 0, st,
                                                    (const T*)logits, V, tokens, parent, depth, row_off, B, node_argmax,
                                                    margin, k_acc, path, bonus, do_accept ? 1 : 0, tickets, partial));
    } else if (do_accept) {
        launch_err = launch_chain(accept_only_kernel, dim3(B), dim3(32), 0, st, tokens, parent, depth, row_off,
                                  (const int32_t*)node_argmax, k_acc, path, bonus);
    }
    return launch_err != cudaSuccess ? launch_err : cudaGetLastError();
}

size_t topk_workspace_bytes() { return align_up(sizeof(unsigned int) * TRJ_MAX_BATCH, 256); }

cudaError_t launch_topk_accept(const void* logits, int32_t dtype, int32_t V, int32_t K,
                               const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                               const int32_t* row_off, int32_t B, int32_t rows_total, int32_t* topk,
                               int32_t* node_argmax, float* margin, int32_t* k_acc, int32_t* path,
                               int32_t* bonus, bool do_accept, void* ws, cudaStream_t st) {
    if (K < 1 || K > TRJ_MAX_TOPK) return cudaErrorInvalidValue;
    count_launch();
    cudaError_t launch_err = cudaSuccess;
    unsigned int* tickets = (unsigned int*)ws;
    if (K == 1) {                                            // the step's arg-max: a kernel of its own, five instructions per element
        DISPATCH_T(dtype, launch_err = launch_chain(argmax_row_accept_kernel<T>, dim3(rows_total), dim3(TOPK_THREADS), 0, st,
                                                    (const T*)logits, V, tokens, parent, depth, row_off, B, node_argmax,
                                                    margin, k_acc, path, bonus, do_accept ? 1 : 0, tickets));
        if (launch_err == cudaSuccess && topk)
            launch_err = cudaMemcpyAsync(topk, node_argmax, sizeof(int32_t) * (size_t)rows_total, cudaMemcpyDeviceToDevice, st);
    } else {
        DISPATCH_T(dtype, launch_err = launch_chain(topk_accept_kernel<T>, dim3(rows_total), dim3(TOPK_THREADS), 0, st,
                                                    (const T*)logits, V, K, tokens, parent, depth, row_off, B, topk, node_argmax,
                                                    margin, k_acc, path, bonus, do_accept ? 1 : 0, tickets));
    }
    return launch_err != cudaSuccess ? launch_err : cudaGetLastError();
}

cudaError_t launch_argmax_table_accept(const TopEntry* table, int32_t entries_per_row, const int32_t* tokens,
                                       const int32_t* parent, const int32_t* depth, const int32_t* row_off, int32_t B,
                                       int32_t rows_total, int32_t* node_argmax, float* margin, int32_t* k_acc,
                                       int32_t* path, int32_t* bonus, bool do_accept, void* ws, cudaStream_t st) {
    count_launch();
    cudaError_t e = launch_chain(argmax_table_accept_kernel, dim3(rows_total), dim3(128), 0, st, table, entries_per_row, tokens,
                                 parent, depth, row_off, B, node_argmax, margin, k_acc, path, bonus, do_accept ? 1 : 0,
                                 (unsigned int*)ws);
    return e != cudaSuccess ? e : cudaGetLastError();
}

// ---------------------------------------------------------------- arg-max + accept without a caller workspace
// Scratch of the allocation-free entry point: the tickets and the per-slice candidates live in this
// file-scope device array, which every GPU that loads the library holds until the process exits.
constexpr int STATIC_MAX_ROWS = TRJ_STATIC_MAX_ROWS;
constexpr size_t STATIC_TICKET_BYTES = 256;
constexpr size_t STATIC_SCRATCH_BYTES = STATIC_TICKET_BYTES + sizeof(Top) * ARGMAX_CHUNKS * (size_t)STATIC_MAX_ROWS;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel can use: the
// device address is looked up once per device (with that device current) and remembered.
static cudaError_t static_scratch_address(void** out, cudaStream_t st) {
    constexpr int MAX_DEVICES = 64;
    static std::mutex mu;
    static void* addr[MAX_DEVICES] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        // the lookup may load the module: it must not happen while `st` is being captured
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        e = cudaStreamIsCapturing(st, &cs);
        if (e != cudaSuccess) return e;
        if (cs != cudaStreamCaptureStatusNone) return cudaErrorStreamCaptureUnsupported;
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        addr[dev] = p;
    }
    *out = addr[dev];
    return cudaSuccess;
}

cudaError_t launch_argmax_accept_static(const void* logits, int32_t dtype, int32_t V,
                                        const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                        const int32_t* row_off, int32_t B, int32_t rows_total,
                                        int32_t* node_argmax, float* margin, int32_t* k_acc, int32_t* path,
                                        int32_t* bonus, cudaStream_t st) {
    void* scratch = nullptr;
    cudaError_t e = static_scratch_address(&scratch, st);
    if (e != cudaSuccess) return e;
    // the array keeps whatever the previous call left: the tickets must start at zero
    e = cudaMemsetAsync(scratch, 0, STATIC_TICKET_BYTES, st);
    if (e != cudaSuccess) return e;
    count_launch();
    unsigned int* tickets = (unsigned int*)scratch;
    Top* partial = (Top*)((char*)scratch + STATIC_TICKET_BYTES);
    dim3 grid(rows_total, ARGMAX_CHUNKS);
    DISPATCH_T(dtype, argmax_accept_kernel<T><<<grid, ARGMAX_THREADS, 0, st>>>(
                          (const T*)logits, V, tokens, parent, depth, row_off, B, node_argmax, margin, k_acc,
                          path, bonus, 1, tickets, partial));
    return cudaGetLastError();
}

cudaError_t launch_compact(void* k_cache, void* v_cache, int32_t L, int32_t B_cache, int32_t B, int32_t H,
                           int32_t max_seq, int32_t D, int32_t dtype, int32_t* seq_len,
                           const int32_t* k_acc, const int32_t* path, cudaStream_t st, unsigned int* tickets) {
    count_launch();
    const int row_vec = (int)(D * dtype_size(dtype) / 16);
    const size_t smem = sizeof(uint4) * COMPACT_BATCH * row_vec;
    cudaError_t e = launch_chain(compact_kernel, dim3(L * B * H * 2), dim3(256), smem, st, (uint4*)k_cache, (uint4*)v_cache,
                                 B_cache, B, H, max_seq, row_vec, seq_len, k_acc, path, tickets);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess || tickets) return e;
    // without a ticket array (the op-level call has no workspace) the lengths are advanced by a second kernel
    count_launch();
    e = launch_chain(advance_len_kernel, dim3((B + 63) / 64), dim3(64), 0, st, seq_len, k_acc, B);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_set_chunk(int32_t* row_off2, int32_t m, cudaStream_t st) {
    count_launch();
    set_chunk_kernel<<<1, 1, 0, st>>>(row_off2, m);
    return cudaGetLastError();
}
cudaError_t launch_prefill_geometry(const int32_t* seq_len_b, int32_t* lens, int32_t n_sub, int32_t sub, int32_t m,
                                    int32_t* off_all, int32_t* off_pieces, cudaStream_t st) {
    count_launch();
    prefill_geometry_kernel<<<1, 32, 0, st>>>(seq_len_b, lens, n_sub, sub, m, off_all, off_pieces);
    return cudaGetLastError();
}
cudaError_t launch_bump_len(int32_t* seq_len_b, int32_t delta, cudaStream_t st) {
    count_launch();
    bump_len_kernel<<<1, 1, 0, st>>>(seq_len_b, delta);
    return cudaGetLastError();
}

}  // namespace trj
