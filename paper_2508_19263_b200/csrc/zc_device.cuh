// Device-side helpers shared by the kernels of libzc.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

#include "zc_bits.cuh"
#include "zc_internal.h"

namespace zc {

constexpr uint32_t kLutEntries = 1u << kLmax;
constexpr size_t kMaxSmem = 227 * 1024;       // usable shared memory per block on sm_100

// Record an error of the call `call_id` unless one of the same call is already there.  True if this
// thread's error is the one that was recorded.
__device__ __forceinline__ bool raise_status(Control* ctl, unsigned long long call_id, uint32_t s)
{
    const unsigned long long mine = (call_id << 8) | s;
    unsigned long long cur = *reinterpret_cast<volatile unsigned long long*>(&ctl->status);
    for (int tries = 0; tries < 64; ++tries) {
        if ((cur >> 8) == call_id && (cur & 0xFF) != 0) return false;
        const unsigned long long old = atomicCAS(&ctl->status, cur, mine);
        if (old == cur) return true;
        cur = old;
    }
    return false;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- development build (-DZC_DEBUG_CHECKS=1; never the shipped library) -------------------------------------------
// Every shared-memory and global-memory access made through the helpers of this header (and the helpers of the
// kernels' own files, which use the same macros) is checked first: a shared address must lie inside the block's shared
// window and be aligned to the access; a global address must lie inside one of the launch's three address ranges
// (readable inputs, writable outputs, workspace; stores only inside the last two) and be aligned.  A violation is
// counted and the access is skipped (loads give zeros): nothing traps, nothing faults, and the host reads the
// counters after the call (zc_test_debug_counts).  One state per translation unit, set by the host before a launch.
#ifndef ZC_DEBUG_CHECKS
#define ZC_DEBUG_CHECKS 0
#endif
#if ZC_DEBUG_CHECKS
struct DebugState {
    unsigned long long lo[3], hi[3];                  // [0] inputs, [1] outputs, [2] workspace
    unsigned int bad_shared, bad_global;
};
static __device__ DebugState g_debug;
__device__ __forceinline__ bool dbg_shared(uint32_t addr, uint32_t bytes)
{
    // the block's shared window ends where its dynamic shared memory ends (static shared memory lies below it)
    extern __shared__ __align__(16) uint8_t zc_dbg_dynamic[];
    uint32_t dyn;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    const uint32_t total = (uint32_t)__cvta_generic_to_shared(zc_dbg_dynamic) + dyn;
    if ((addr & (bytes - 1)) == 0 && addr + bytes <= total) return true;
    atomicAdd(&g_debug.bad_shared, 1u);
    return false;
}
__device__ __forceinline__ bool dbg_global(const void* p, uint32_t bytes, uint32_t align, bool store)
{
    const unsigned long long a = (unsigned long long)p;
    bool ok = false;
    for (int k = store ? 1 : 0; k < 3; ++k) ok = ok || (a >= g_debug.lo[k] && a + bytes <= g_debug.hi[k]);
    ok = ok && (a & (align - 1)) == 0;
    if (!ok) atomicAdd(&g_debug.bad_global, 1u);
    return ok;
}
#define ZC_DBG_SHARED(addr, bytes, fail) do { if (!dbg_shared((addr), (bytes))) { fail; } } while (0)
#define ZC_DBG_GLOBAL(p, bytes, align, store, fail) do { if (!dbg_global((p), (bytes), (align), (store))) { fail; } } while (0)
// host: the address ranges of the launch that follows on `st` (pairs of first byte and byte count)
inline void dbg_set_ranges(cudaStream_t st, const void* in, size_t in_bytes, const void* out, size_t out_bytes,
                           const void* ws, size_t ws_bytes)
{
    DebugState h{};
    const void* lo[3] = {in, out, ws};
    const size_t n[3] = {in_bytes, out_bytes, ws_bytes};
    for (int k = 0; k < 3; ++k) { h.lo[k] = (unsigned long long)lo[k]; h.hi[k] = h.lo[k] + n[k]; }
    cudaMemcpyToSymbolAsync(g_debug, &h, 6 * sizeof(unsigned long long), 0, cudaMemcpyHostToDevice, st);
}
inline void dbg_read_counts(uint32_t out[2])
{
    DebugState h{};
    cudaDeviceSynchronize();
    if (cudaMemcpyFromSymbol(&h, g_debug, sizeof h) == cudaSuccess) { out[0] += h.bad_shared; out[1] += h.bad_global; }
    const unsigned int zero[2] = {0, 0};
    cudaMemcpyToSymbol(g_debug, zero, sizeof zero, offsetof(DebugState, bad_shared));
}
// the hull of several buffers (a batched launch): smallest first byte, largest last byte
struct DbgHull {
    unsigned long long lo = ~0ull, hi = 0;
    void add(const void* p, size_t n) { if (p && n) { lo = std::min<unsigned long long>(lo, (unsigned long long)p); hi = std::max<unsigned long long>(hi, (unsigned long long)p + n); } }
    const void* ptr() const { return hi ? (const void*)lo : nullptr; }
    size_t bytes() const { return hi ? (size_t)(hi - lo) : 0; }
};
#else
#define ZC_DBG_SHARED(addr, bytes, fail) do { } while (0)
#define ZC_DBG_GLOBAL(p, bytes, align, store, fail) do { } while (0)
#endif


__device__ __forceinline__ uint4 ld_nc_v4(const void* p)
{
    ZC_DBG_GLOBAL(p, 16, 16, false, return make_uint4(0, 0, 0, 0));
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ld_nc_v2(const void* p)
{
    ZC_DBG_GLOBAL(p, 8, 8, false, return make_uint2(0, 0));
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_cs_v4(void* p, uint4 v)
{
    ZC_DBG_GLOBAL(p, 16, 16, true, return);
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// 32-byte store (one full sector per lane); the address must be 32-byte aligned
__device__ __forceinline__ void st_cs_v8(void* p, const uint32_t v[8])
{
    ZC_DBG_GLOBAL(p, 32, 32, true, return);
    asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}
__device__ __forceinline__ void st_cs_v2(void* p, uint2 v)
{
    ZC_DBG_GLOBAL(p, 8, 8, true, return);
    asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" :: "l"(p), "r"(v.x), "r"(v.y) : "memory");
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    ZC_DBG_SHARED(addr, 4, return 0);
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts8(uint32_t addr, uint32_t v)
{
    ZC_DBG_SHARED(addr, 1, return);
    asm volatile("st.shared.u8 [%0], %1;" :: "r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v)
{
    ZC_DBG_SHARED(addr, 4, return);
    asm volatile("st.shared.u32 [%0], %1;" :: "r"(addr), "r"(v) : "memory");
}

// Load up to 16 bytes that may run past the end of the input: missing bytes read as zero.
__device__ __forceinline__ uint4 load16_guarded(const uint8_t* base, uint64_t off, uint64_t limit)
{
    if (off + 16 <= limit) return ld_nc_v4(base + off);
    uint32_t w[4] = {0, 0, 0, 0};
    for (uint32_t i = 0; i < 16 && off + i < limit; ++i) w[i >> 2] |= (uint32_t)base[off + i] << (8 * (i & 3));
    return make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait for a phase of an mbarrier; false when the wait gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t spin_limit)
{
    for (uint32_t spins = 0; spins <= spin_limit; ++spins)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// Bulk asynchronous copy global -> shared of this CTA, completion counted in bytes on an mbarrier.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar)
{
    ZC_DBG_GLOBAL(src, bytes, 16, false, return); ZC_DBG_SHARED(smem_u32(dst), 16, return); ZC_DBG_SHARED(smem_u32(dst) + bytes - 16, 16, return);
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}


// the same with the destination given as a shared address
__device__ __forceinline__ void bulk_g2s_addr(uint32_t dst_s, const void* src, uint32_t bytes, uint64_t* bar)
{
    ZC_DBG_GLOBAL(src, bytes, 16, false, return); ZC_DBG_SHARED(dst_s, 16, return); ZC_DBG_SHARED(dst_s + bytes - 16, 16, return);
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst_s), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

inline int sm_count()
{
    static int cached = 0;
    if (!cached) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
        cached = n;
    }
    return cached;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace zc
