// Split + histogram kernels and zc_histogram, zc_histogram_batch (and their XOR-delta forms).
//
// Delta form (Sec. 3.1 / 4.1, delta checkpoints): when a base tensor is given, what is counted is the
// bitwise XOR of the input with the base, computed on the fly in registers.
#include "zc_device.cuh"

namespace zc {

constexpr int kHistThreads = 512;

// ------------------------------------------------------------------------------------------------
// split + histogram
// ------------------------------------------------------------------------------------------------
// Each lane of a warp owns its own copy of every bin (bins[stream][symbol][lane]): the bank of an
// update is the lane number, so updates of one warp never collide, however skewed the exponent
// distribution is.  The 64 KiB of bins are shared by the warps of the block through shared atomics.

__device__ __forceinline__ void red_add1(uint32_t addr)
{
    ZC_DBG_SHARED(addr, 4, return);
    asm volatile("red.shared.add.u32 [%0], 1;" :: "r"(addr) : "memory");
}

// Count the 8 + 8 symbols of one 16-byte group.  lane_bins = shared address of bins[0][0][lane];
// a symbol's counter is 128 bytes further per symbol value, stream 1 starts 32 KiB later.
template <int FMT>
__device__ __forceinline__ void count16(const uint4 x, uint32_t lane_bins)
{
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
    uint32_t e[2], sm[2];
    split16<FMT>(w, e, sm);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t a = __byte_perm(e[h], 0, 0x4440 + q);
            const uint32_t b = __byte_perm(sm[h], 0, 0x4440 + q);
            red_add1(lane_bins + a * 128u);
            red_add1(lane_bins + 32768u + b * 128u);
        }
    }
}

__device__ __forceinline__ uint4 xor4(const uint4 a, const uint4 b) { return make_uint4(a.x ^ b.x, a.y ^ b.y, a.z ^ b.z, a.w ^ b.w); }

template <int FMT>
__global__ void __launch_bounds__(kHistThreads)
hist_kernel(const uint8_t* __restrict__ in, const uint8_t* __restrict__ base, uint64_t input_bytes, uint64_t n_syms,
            unsigned long long* __restrict__ hist)
{
    extern __shared__ uint32_t bins[];           // [2][256][32]
    const uint32_t lane = threadIdx.x & 31;
    for (uint32_t i = threadIdx.x; i < 2 * 256 * 32; i += kHistThreads) bins[i] = 0;
    __syncthreads();
    const uint32_t lane_bins = smem_u32(bins) + 4 * lane;

    // groups of 16 input bytes = 8 symbols of each stream; complete groups first, four loads in flight
    const uint64_t n_full = n_syms / 8 < input_bytes / 16 ? n_syms / 8 : input_bytes / 16;
    const uint64_t stride = (uint64_t)gridDim.x * kHistThreads;
    uint64_t v = (uint64_t)blockIdx.x * kHistThreads + threadIdx.x;
    if (base) {
        for (; v + stride < n_full; v += 2 * stride) {          // two pairs of loads in flight
            const uint4 x0 = ld_nc_v4(in + 16 * v), y0 = ld_nc_v4(base + 16 * v);
            const uint4 x1 = ld_nc_v4(in + 16 * (v + stride)), y1 = ld_nc_v4(base + 16 * (v + stride));
            count16<FMT>(xor4(x0, y0), lane_bins);
            count16<FMT>(xor4(x1, y1), lane_bins);
        }
        for (; v < n_full; v += stride) count16<FMT>(xor4(ld_nc_v4(in + 16 * v), ld_nc_v4(base + 16 * v)), lane_bins);
    }
    for (; v + 3 * stride < n_full; v += 4 * stride) {
        const uint4 x0 = ld_nc_v4(in + 16 * v);
        const uint4 x1 = ld_nc_v4(in + 16 * (v + stride));
        const uint4 x2 = ld_nc_v4(in + 16 * (v + 2 * stride));
        const uint4 x3 = ld_nc_v4(in + 16 * (v + 3 * stride));
        count16<FMT>(x0, lane_bins);
        count16<FMT>(x1, lane_bins);
        count16<FMT>(x2, lane_bins);
        count16<FMT>(x3, lane_bins);
    }
    for (; v < n_full; v += stride) count16<FMT>(ld_nc_v4(in + 16 * v), lane_bins);
    // the ragged last group (fewer than 8 symbols, or input bytes that end inside the group)
    if (blockIdx.x == 0 && threadIdx.x == 0 && 8 * n_full < n_syms) {
        uint4 x = load16_guarded(in, 16 * n_full, input_bytes);
        if (base) x = xor4(x, load16_guarded(base, 16 * n_full, input_bytes));
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
        uint32_t e[2], sm[2];
        split16<FMT>(w, e, sm);
        const uint32_t nv = (uint32_t)(n_syms - 8 * n_full);
        for (uint32_t i = 0; i < nv && i < 8; ++i) {
            const uint32_t a = (e[i >> 2] >> (8 * (i & 3))) & 0xFF;
            const uint32_t b = (sm[i >> 2] >> (8 * (i & 3))) & 0xFF;
            atomicAdd(&bins[a * 32 + lane], 1u);
            atomicAdd(&bins[(256 + b) * 32 + lane], 1u);
        }
    }
    __syncthreads();
    for (uint32_t b = threadIdx.x; b < 512; b += kHistThreads) {
        uint32_t sum = 0;
#pragma unroll 8
        for (uint32_t i = 0; i < 32; ++i) sum += bins[b * 32 + ((i + lane) & 31)];
        if (sum) atomicAdd(&hist[b], (unsigned long long)sum);
    }
}

// Many tensors per launch.  The complete 16-byte groups of all tensors form one index space that is cut into
// equal contiguous ranges, one per block; a block adds its bins to a tensor's histogram whenever its range
// moves on to the next tensor.  Ragged last groups are counted straight into global memory.
struct HistItem {
    const uint8_t* in;
    const uint8_t* base;                         // XOR-delta form: the tensor the input is XOR-ed with, or null
    uint64_t input_bytes, n_syms;
    uint64_t first_vec;                          // complete groups of all earlier tensors of the launch
};
constexpr uint32_t kHistBatchMax = 768;          // keeps the parameter block below 32 KiB
struct HistBatchParams {
    unsigned long long* hist;                    // [n_tensors][2][256]
    uint64_t total_vec;
    uint32_t n_tensors, pad;
    HistItem item[kHistBatchMax];
};
static_assert(sizeof(HistBatchParams) < 32764, "kernel parameters are limited to 32764 bytes");

template <int FMT>
__global__ void __launch_bounds__(kHistThreads)
hist_batch_kernel(const __grid_constant__ HistBatchParams B)
{
    extern __shared__ uint32_t bins[];           // [2][256][32]
    const uint32_t lane = threadIdx.x & 31;
    for (uint32_t i = threadIdx.x; i < 2 * 256 * 32; i += kHistThreads) bins[i] = 0;
    const uint32_t lane_bins = smem_u32(bins) + 4 * lane;

    // ragged last groups (fewer than 8 symbols, or input bytes that end inside the group): one thread each
    if (threadIdx.x == 0) {
        for (uint32_t t = blockIdx.x; t < B.n_tensors; t += gridDim.x) {
            const HistItem& I = B.item[t];
            const uint64_t n_full = I.n_syms / 8 < I.input_bytes / 16 ? I.n_syms / 8 : I.input_bytes / 16;
            if (8 * n_full >= I.n_syms) continue;
            uint4 x = load16_guarded(I.in, 16 * n_full, I.input_bytes);
            if (I.base) x = xor4(x, load16_guarded(I.base, 16 * n_full, I.input_bytes));
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
            uint32_t e[2], sm[2];
            split16<FMT>(w, e, sm);
            const uint32_t nv = (uint32_t)(I.n_syms - 8 * n_full);
            for (uint32_t i = 0; i < nv && i < 8; ++i) {
                const uint32_t a = (e[i >> 2] >> (8 * (i & 3))) & 0xFF;
                const uint32_t b = (sm[i >> 2] >> (8 * (i & 3))) & 0xFF;
                atomicAdd(&B.hist[512ull * t + a], 1ull);
                atomicAdd(&B.hist[512ull * t + 256 + b], 1ull);
            }
        }
    }
    __syncthreads();

    uint64_t v_lo = (uint64_t)blockIdx.x * B.total_vec / gridDim.x;
    const uint64_t v_hi = (uint64_t)(blockIdx.x + 1) * B.total_vec / gridDim.x;
    if (v_lo >= v_hi) return;
    // the last tensor that starts at or before v_lo (tensors without complete groups share their start with the next)
    uint32_t lo = 0, hi = B.n_tensors;
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) / 2;
        if (B.item[mid].first_vec <= v_lo) lo = mid; else hi = mid;
    }
    for (uint32_t t = lo; t < B.n_tensors && v_lo < v_hi; ++t) {
        const uint64_t first = B.item[t].first_vec;
        const uint64_t end = t + 1 < B.n_tensors ? B.item[t + 1].first_vec : B.total_vec;
        if (v_lo >= end) continue;
        const uint8_t* in = B.item[t].in;
        const uint8_t* base = B.item[t].base;
        const uint64_t seg_hi = (v_hi < end ? v_hi : end) - first;
        uint64_t v = v_lo - first + threadIdx.x;
        constexpr uint64_t stride = kHistThreads;
        if (base) {
            for (; v + stride < seg_hi; v += 2 * stride) {       // two pairs of loads in flight
                const uint4 x0 = ld_nc_v4(in + 16 * v), y0 = ld_nc_v4(base + 16 * v);
                const uint4 x1 = ld_nc_v4(in + 16 * (v + stride)), y1 = ld_nc_v4(base + 16 * (v + stride));
                count16<FMT>(xor4(x0, y0), lane_bins);
                count16<FMT>(xor4(x1, y1), lane_bins);
            }
            for (; v < seg_hi; v += stride) count16<FMT>(xor4(ld_nc_v4(in + 16 * v), ld_nc_v4(base + 16 * v)), lane_bins);
        }
        for (; v + 3 * stride < seg_hi; v += 4 * stride) {       // four loads in flight
            const uint4 x0 = ld_nc_v4(in + 16 * v);
            const uint4 x1 = ld_nc_v4(in + 16 * (v + stride));
            const uint4 x2 = ld_nc_v4(in + 16 * (v + 2 * stride));
            const uint4 x3 = ld_nc_v4(in + 16 * (v + 3 * stride));
            count16<FMT>(x0, lane_bins);
            count16<FMT>(x1, lane_bins);
            count16<FMT>(x2, lane_bins);
            count16<FMT>(x3, lane_bins);
        }
        for (; v < seg_hi; v += stride) count16<FMT>(ld_nc_v4(in + 16 * v), lane_bins);
        __syncthreads();
        // add the bins to this tensor's histogram and clear them for the next one
        for (uint32_t b = threadIdx.x; b < 512; b += kHistThreads) {
            uint32_t sum = 0;
#pragma unroll 8
            for (uint32_t i = 0; i < 32; ++i) {
                const uint32_t k = b * 32 + ((i + lane) & 31);
                sum += bins[k];
                bins[k] = 0;
            }
            if (sum) atomicAdd(&B.hist[512ull * t + b], (unsigned long long)sum);
        }
        __syncthreads();
        v_lo = first + seg_hi;
    }
}

}  // namespace zc

namespace zc {
void debug_counts_hist(uint32_t out[2])
{
#if ZC_DEBUG_CHECKS
    dbg_read_counts(out);
#else
    (void)out;
#endif
}
}  // namespace zc

using namespace zc;

extern "C" {

zc_status zc_histogram(const zc_plan_t* p, const void* d_in, uint64_t* d_hist, void* cuda_stream)
{
    return zc_histogram_xor(p, d_in, nullptr, d_hist, cuda_stream);
}

zc_status zc_histogram_xor(const zc_plan_t* p, const void* d_in, const void* d_base, uint64_t* d_hist, void* cuda_stream)
{
    if (!p || !d_hist || (!d_in && p->n_elems) || !aligned16(d_in) || !aligned16(d_base)) return ZC_E_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(d_hist, 0, 2 * 256 * sizeof(uint64_t), st) != cudaSuccess) return ZC_E_CUDA;
    if (p->n_syms == 0) return ZC_OK;
    const size_t smem = 2 * 256 * 32 * sizeof(uint32_t);
    const uint64_t n_vec = (p->n_syms + 7) / 8;
    const uint64_t want = (n_vec + kHistThreads * 8 - 1) / (kHistThreads * 8);
    const uint32_t grid = (uint32_t)std::min<uint64_t>(std::max<uint64_t>(want, 1), (uint64_t)sm_count() * 3);
    cudaError_t e = cudaSuccess;
    auto launch = [&](auto kern) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return;
#if ZC_DEBUG_CHECKS
        DbgHull rd;
        rd.add(d_in, p->input_bytes);
        rd.add(d_base, p->input_bytes);
        dbg_set_ranges(st, rd.ptr(), rd.bytes(), d_hist, 2 * 256 * sizeof(uint64_t), nullptr, 0);
#endif
        kern<<<grid, kHistThreads, smem, st>>>((const uint8_t*)d_in, (const uint8_t*)d_base, p->input_bytes, p->n_syms,
                                                (unsigned long long*)d_hist);
        e = cudaGetLastError();
    };
    switch (p->format) {
    case ZC_FMT_BF16: launch(hist_kernel<ZC_FMT_BF16>); break;
    case ZC_FMT_FP8_E4M3: case ZC_FMT_FP8_E5M2: launch(hist_kernel<ZC_FMT_FP8_E4M3>); break;
    case ZC_FMT_SCALE_U8: launch(hist_kernel<ZC_FMT_SCALE_U8>); break;
    default: launch(hist_kernel<ZC_FMT_FP4_E2M1>); break;
    }
    return e == cudaSuccess ? ZC_OK : ZC_E_CUDA;
}

zc_status zc_histogram_batch(uint32_t n_tensors, const zc_plan_t* const* plans, const void* const* d_in, uint64_t* d_hists,
                             void* cuda_stream)
{
    return zc_histogram_batch_xor(n_tensors, plans, d_in, nullptr, d_hists, cuda_stream);
}

zc_status zc_histogram_batch_xor(uint32_t n_tensors, const zc_plan_t* const* plans, const void* const* d_in,
                                 const void* const* d_base, uint64_t* d_hists, void* cuda_stream)
{
    if (n_tensors == 0) return ZC_OK;
    if (!plans || !d_in || !d_hists) return ZC_E_INVALID_ARG;
    for (uint32_t t = 0; t < n_tensors; ++t) {
        if (!plans[t] || (!d_in[t] && plans[t]->n_elems) || !aligned16(d_in[t])) return ZC_E_INVALID_ARG;
        if (d_base && !aligned16(d_base[t])) return ZC_E_INVALID_ARG;
        if (plans[t]->format != plans[0]->format) return ZC_E_INVALID_ARG;
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(d_hists, 0, (size_t)n_tensors * 2 * 256 * sizeof(uint64_t), st) != cudaSuccess) return ZC_E_CUDA;
    const size_t smem = 2 * 256 * 32 * sizeof(uint32_t);
    static thread_local HistBatchParams B;
    for (uint32_t base = 0; base < n_tensors; base += kHistBatchMax) {
        const uint32_t n = std::min<uint32_t>(kHistBatchMax, n_tensors - base);
        uint64_t total = 0, any_syms = 0;
        for (uint32_t i = 0; i < n; ++i) {
            const zc_plan_t* p = plans[base + i];
            B.item[i].in = (const uint8_t*)d_in[base + i];
            B.item[i].base = d_base ? (const uint8_t*)d_base[base + i] : nullptr;
            B.item[i].input_bytes = p->input_bytes;
            B.item[i].n_syms = p->n_syms;
            B.item[i].first_vec = total;
            total += std::min<uint64_t>(p->n_syms / 8, p->input_bytes / 16);
            any_syms += p->n_syms;
        }
        if (any_syms == 0) continue;
        B.hist = (unsigned long long*)d_hists + 512ull * base;
        B.total_vec = total;
        B.n_tensors = n;
        B.pad = 0;
        const uint64_t want = (total + kHistThreads * 8 - 1) / (kHistThreads * 8);
        const uint32_t grid = (uint32_t)std::min<uint64_t>(std::max<uint64_t>(want, 1), (uint64_t)sm_count() * 3);
        cudaError_t e = cudaSuccess;
        auto launch = [&](auto kern) {
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return;
#if ZC_DEBUG_CHECKS
            DbgHull rd;
            for (uint32_t i = 0; i < n; ++i) { rd.add(B.item[i].in, B.item[i].input_bytes); rd.add(B.item[i].base, B.item[i].input_bytes); }
            dbg_set_ranges(st, rd.ptr(), rd.bytes(), B.hist, (size_t)n * 2 * 256 * sizeof(uint64_t), nullptr, 0);
#endif
            kern<<<grid, kHistThreads, smem, st>>>(B);
            e = cudaGetLastError();
        };
        switch (plans[0]->format) {
        case ZC_FMT_BF16: launch(hist_batch_kernel<ZC_FMT_BF16>); break;
        case ZC_FMT_FP8_E4M3: case ZC_FMT_FP8_E5M2: launch(hist_batch_kernel<ZC_FMT_FP8_E4M3>); break;
        case ZC_FMT_SCALE_U8: launch(hist_batch_kernel<ZC_FMT_SCALE_U8>); break;
        default: launch(hist_batch_kernel<ZC_FMT_FP4_E2M1>); break;
        }
        if (e != cudaSuccess) return ZC_E_CUDA;
    }
    return ZC_OK;
}

}  // extern "C"
