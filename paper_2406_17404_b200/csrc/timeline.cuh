// Optional clock stamps of the per-layer kernels (compiled in with -DTRJ_TIMELINE only; the default build has none of
// it).  Every instrumented launch records, in a table of its translation unit, the time its first CTA got past the
// wait for its predecessor ("release") and the time its last CTA ended.  Launches of one kind are numbered in the
// order they complete, which is their launch order because two launches of one kind never overlap in a step.
#pragma once
#include <stdint.h>

#ifdef TRJ_TIMELINE
namespace trj {
namespace tl {

constexpr int KINDS = 6;          // see TRJ_TL_* in trj.h
constexpr int SLOTS = 512;        // launches of one kind between two resets
struct Rec { unsigned long long begin_inv, end; unsigned int done, pad; };   // begin_inv = ~(earliest release): zero = none yet
static __device__ Rec g_rec[KINDS][SLOTS];
static __device__ unsigned int g_count[KINDS];
static __device__ int g_sm_now[256];      // CTAs of this translation unit's projection kernels resident on each SM right now
static __device__ int g_sm_peak;          // ... and the most that were ever resident on one SM at the same time

__device__ __forceinline__ unsigned long long now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// First and last thing a CTA does (one thread): how many CTAs of the kernel share an SM.
__device__ __forceinline__ unsigned int smid() {
    unsigned int s;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(s));
    return s;
}
__device__ __forceinline__ void enter() { atomicMax(&g_sm_peak, atomicAdd(&g_sm_now[smid() & 255u], 1) + 1); }
__device__ __forceinline__ void leave() { atomicSub(&g_sm_now[smid() & 255u], 1); }
inline int sm_peak() {
    int v = -1;
    if (cudaMemcpyFromSymbol(&v, g_sm_peak, sizeof(int)) != cudaSuccess) return -1;
    return v;
}
// One thread per CTA, right after the CTA's wait for the previous kernel.
__device__ __forceinline__ unsigned int begin(int kind) {
    unsigned int c = *(volatile unsigned int*)&g_count[kind];
    if (c >= SLOTS) c = SLOTS - 1;
    atomicMax(&g_rec[kind][c].begin_inv, ~now());
    return c;
}
// The same thread, as the last thing the CTA does.
__device__ __forceinline__ void end(int kind, unsigned int c) {
    atomicMax(&g_rec[kind][c].end, now());
    __threadfence();
    if (atomicAdd(&g_rec[kind][c].done, 1u) + 1u == gridDim.x * gridDim.y * gridDim.z) atomicAdd(&g_count[kind], 1u);
}
inline cudaError_t reset(cudaStream_t st) {
    void *rec = nullptr, *cnt = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&rec, g_rec);
    if (e == cudaSuccess) e = cudaGetSymbolAddress(&cnt, g_count);
    if (e == cudaSuccess) e = cudaMemsetAsync(rec, 0, sizeof(Rec) * KINDS * SLOTS, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(cnt, 0, sizeof(unsigned int) * KINDS, st);
    return e;
}
// Launches of `kind` recorded in this translation unit since the last reset: begin / end in ns; returns their number.
inline int read(int kind, int max_launches, uint64_t* begin_ns, uint64_t* end_ns) {
    static Rec host[SLOTS];
    unsigned int counts[KINDS];
    if (cudaMemcpyFromSymbol(counts, g_count, sizeof(counts)) != cudaSuccess) return -1;
    if (cudaMemcpyFromSymbol(host, g_rec, sizeof(Rec) * SLOTS, sizeof(Rec) * SLOTS * (size_t)kind) != cudaSuccess) return -1;
    int n = (int)counts[kind];
    if (n > SLOTS) n = SLOTS;
    if (n > max_launches) n = max_launches;
    for (int i = 0; i < n; ++i) { begin_ns[i] = ~host[i].begin_inv; end_ns[i] = host[i].end; }
    return n;
}

}  // namespace tl
}  // namespace trj
#define TRJ_TL_ENTER() do { if (threadIdx.x == 0) ::trj::tl::enter(); } while (0)
#define TRJ_TL_LEAVE() do { if (threadIdx.x == 0) ::trj::tl::leave(); } while (0)
#define TRJ_TL_DECL unsigned int tl_slot__ = 0
#define TRJ_TL_BEGIN(kind) do { if (threadIdx.x == 0) tl_slot__ = ::trj::tl::begin(kind); } while (0)
#define TRJ_TL_END(kind) do { if (threadIdx.x == 0) ::trj::tl::end(kind, tl_slot__); } while (0)
#else
#define TRJ_TL_ENTER()
#define TRJ_TL_LEAVE()
#define TRJ_TL_DECL
#define TRJ_TL_BEGIN(kind)
#define TRJ_TL_END(kind)
#endif
