// sm_100a kernels of libzc and the C-ABI entry points that launch them.
//
//   hist_kernel    split + histogram            (zc_histogram)
//   encode_kernel  split + length scan + pack   (zc_compress)    one warp per chunk, one lane per subchunk
//   decode_kernel  table decode + merge         (zc_decompress)  one warp per chunk, one lane per subchunk
//
// None of this is a contraction, so no tensor cores: the kernels are bounded by HBM traffic, by the
// integer pipes and by shared-memory latency of the per-symbol table lookups.
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

#include "zc_bits.cuh"
#include "zc_internal.h"

namespace zc {

constexpr int kHistThreads = 256;
constexpr uint32_t kSpinLimit = 1u << 22;     // bounded waits: look-back and mbarrier
constexpr uint32_t kLutEntries = 1u << kLmax;

// ------------------------------------------------------------------------------------------------
// small device helpers
// ------------------------------------------------------------------------------------------------

__device__ __forceinline__ void raise_status(Control* ctl, uint32_t s) { atomicCAS(&ctl->status, 0u, s); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint4 ld_nc_v4(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ld_nc_v2(const void* p)
{
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_cs_v4(void* p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void st_cs_v2(void* p, uint2 v)
{
    asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" :: "l"(p), "r"(v.x), "r"(v.y) : "memory");
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts8(uint32_t addr, uint32_t v)
{
    asm volatile("st.shared.u8 [%0], %1;" :: "r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v)
{
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

// ------------------------------------------------------------------------------------------------
// split + histogram
// ------------------------------------------------------------------------------------------------
// Each lane of a warp owns its own copy of every bin (bins[stream][symbol][lane]): the bank of an
// update is the lane number, so updates of one warp never collide, however skewed the exponent
// distribution is.  The 64 KiB of bins are shared by the warps of the block through shared atomics.

template <int FMT>
__global__ void __launch_bounds__(kHistThreads)
hist_kernel(const uint8_t* __restrict__ in, uint64_t input_bytes, uint64_t n_syms, unsigned long long* __restrict__ hist)
{
    extern __shared__ uint32_t bins[];           // [2][256][32]
    const uint32_t lane = threadIdx.x & 31;
    for (uint32_t i = threadIdx.x; i < 2 * 256 * 32; i += kHistThreads) bins[i] = 0;
    __syncthreads();

    const uint64_t n_vec = (n_syms + 7) / 8;     // 16 input bytes = 8 symbols of each stream
    for (uint64_t v = (uint64_t)blockIdx.x * kHistThreads + threadIdx.x; v < n_vec; v += (uint64_t)gridDim.x * kHistThreads) {
        const uint4 x = load16_guarded(in, 16 * v, input_bytes);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
        uint32_t e[2], sm[2];
        split16<FMT>(w, e, sm);
        const uint64_t left = n_syms - 8 * v;
        const uint32_t nv = left < 8 ? (uint32_t)left : 8u;
        if (nv == 8) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t a = (e[i >> 2] >> (8 * (i & 3))) & 0xFF;
                const uint32_t b = (sm[i >> 2] >> (8 * (i & 3))) & 0xFF;
                atomicAdd(&bins[a * 32 + lane], 1u);
                atomicAdd(&bins[(256 + b) * 32 + lane], 1u);
            }
        } else {
            for (uint32_t i = 0; i < nv; ++i) {
                const uint32_t a = (e[i >> 2] >> (8 * (i & 3))) & 0xFF;
                const uint32_t b = (sm[i >> 2] >> (8 * (i & 3))) & 0xFF;
                atomicAdd(&bins[a * 32 + lane], 1u);
                atomicAdd(&bins[(256 + b) * 32 + lane], 1u);
            }
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

// ------------------------------------------------------------------------------------------------
// encoder
// ------------------------------------------------------------------------------------------------

struct EncTables { uint32_t enc[2][256]; };     // (length << 16) | code value; 0 = symbol has no code

struct EncParams {
    const uint8_t* in;
    uint8_t* out;
    Control* ctl;
    unsigned long long* flags;                   // one look-back word per chunk
    uint64_t input_bytes, n_syms, n_elems;
    uint32_t n_chunks, cs, sub, chunk_bytes;     // symbols per chunk / per subchunk
    uint32_t mode[2];
    uint32_t format, group;
    Layout lay;
    uint32_t stage_stride;                       // bytes of one stream's symbol staging per warp
    uint32_t sub_magic;                          // ceil(2^32 / sub): k / sub == umulhi(k, sub_magic) for k < 2^17
};

constexpr unsigned long long kFlagAggregate = 1ull << 62, kFlagPrefix = 2ull << 62, kFlagValue = (1ull << 62) - 1;

__device__ __forceinline__ unsigned long long ld_flag(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_flag(unsigned long long* p, unsigned long long v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}

// Sum of the sizes (16-byte units) of all chunks before chunk c: single-pass look-back over the
// per-chunk words that earlier chunks publish.  Chunks are handed out in increasing order by a
// ticket, so every predecessor is already running or finished.  Returns false if a wait gave up.
__device__ bool lookback_exclusive(unsigned long long* flags, uint32_t c, uint32_t lane, uint64_t own, uint64_t& excl)
{
    if (c == 0) {
        if (lane == 0) st_flag(&flags[0], kFlagPrefix | own);
        excl = 0;
        return true;
    }
    if (lane == 0) st_flag(&flags[c], kFlagAggregate | own);
    uint64_t sum = 0;
    int64_t base = (int64_t)c - 1;               // lane i looks at chunk base - i
    uint32_t spins = 0;
    while (true) {
        const int64_t idx = base - lane;
        unsigned long long f = kFlagPrefix;      // before chunk 0: prefix 0
        if (idx >= 0) f = ld_flag(&flags[idx]);
        const uint32_t ready = __ballot_sync(0xFFFFFFFFu, (f >> 62) != 0);
        const uint32_t prefix = __ballot_sync(0xFFFFFFFFu, (f >> 62) == 2);
        // usable lanes: from lane 0 up to the first one holding a prefix, all of them ready
        const uint32_t first_prefix = prefix ? (uint32_t)__ffs(prefix) - 1 : 32u;
        const uint32_t need = first_prefix == 32 ? 0xFFFFFFFFu : (0xFFFFFFFFu >> (31 - first_prefix));
        if ((ready & need) != need) {
            if (++spins > kSpinLimit) return false;
            __nanosleep(64);
            continue;
        }
        uint64_t v = (lane <= first_prefix || first_prefix == 32) ? (f & kFlagValue) : 0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        sum += v;
        if (first_prefix != 32) break;
        base -= 32;
    }
    excl = sum;
    if (lane == 0) st_flag(&flags[c], kFlagPrefix | (sum + own));
    return true;
}

// Symbol k of a chunk is staged at byte k + 4 * (k / sub): subchunk regions are padded by 4 bytes
// so that lanes walking their own regions hit different banks.

template <int FMT>
__global__ void __launch_bounds__(512)
encode_kernel(const __grid_constant__ EncParams P, const __grid_constant__ EncTables T)
{
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const bool huff0 = P.mode[0] == ZC_MODE_HUFF, huff1 = P.mode[1] == ZC_MODE_HUFF;
    const uint32_t n_huff = (huff0 ? 1u : 0u) + (huff1 ? 1u : 0u);

    // shared: enc[2][256] | per warp: sub_bits[2][32] | per warp: staging[n_huff][stage_stride]
    uint32_t* enc = reinterpret_cast<uint32_t*>(smem);
    uint32_t* sub_bits_all = enc + 512;
    uint8_t* stage_all = reinterpret_cast<uint8_t*>(sub_bits_all + 64 * n_warps);
    for (uint32_t i = threadIdx.x; i < 512; i += blockDim.x) enc[i] = T.enc[i >> 8][i & 255];
    uint32_t* sub_bits = sub_bits_all + 64 * warp;
    uint8_t* stage = stage_all + (size_t)warp * n_huff * P.stage_stride;

    // block 0 writes the static parts of the table sections and the tail padding of raw bodies
    if (blockIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            if (P.mode[s] == ZC_MODE_HUFF) {
                for (uint32_t v = threadIdx.x; v < 256; v += blockDim.x) P.out[P.lay.section_off[s] + v] = (uint8_t)(T.enc[s][v] >> 16);
                const uint32_t padded = (P.n_chunks + 3) & ~3u;
                for (uint32_t i = P.n_chunks + threadIdx.x; i < padded; i += blockDim.x)
                    reinterpret_cast<uint32_t*>(P.out + P.lay.chunk_off_tab[s])[i] = 0;
            } else {
                const uint64_t lo = (P.n_syms + 7) & ~7ull, hi = (P.n_syms + 15) & ~15ull;
                for (uint64_t i = lo + threadIdx.x; i < hi; i += blockDim.x) P.out[P.lay.section_off[s] + i] = 0;
            }
        }
    }
    __syncthreads();

    uint32_t first_bad = 0;
    while (true) {
        uint32_t c = 0;
        if (lane == 0) c = atomicAdd(&P.ctl->ticket, 1u);
        c = __shfl_sync(0xFFFFFFFFu, c, 0);
        if (c >= P.n_chunks) break;
        const uint64_t c_lo = (uint64_t)c * P.cs;
        const uint32_t c_syms = (uint32_t)min((uint64_t)P.cs, P.n_syms - c_lo);

        sub_bits[lane] = 0;
        sub_bits[32 + lane] = 0;
        __syncwarp();

        // ---- phase A: coalesced load, split, raw stores, symbol staging, code-length sums ----
        const uint32_t n_vec = (c_syms + 7) / 8;
        for (uint32_t it = lane; it < n_vec; it += 32) {
            const uint32_t k = it * 8;
            const uint4 x = load16_guarded(P.in, 2 * (c_lo + k), P.input_bytes);
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
            uint32_t sy[2][2];
            split16<FMT>(w, sy[0], sy[1]);
            const uint32_t nv = min(8u, c_syms - k);
            uint32_t hs = 0;
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                if (P.mode[s] == ZC_MODE_RAW) {
                    st_cs_v2(P.out + P.lay.section_off[s] + c_lo + k, make_uint2(sy[s][0], sy[s][1]));
                } else {
                    uint32_t acc = 0, bad = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t v = (sy[s][i >> 2] >> (8 * (i & 3))) & 0xFF;
                        const uint32_t e = (uint32_t)i < nv ? enc[256 * s + v] : 0x10000u;
                        bad |= (e == 0);
                        acc += e;
                    }
                    if (bad) first_bad = ZC_E_NO_CODE;
                    const uint32_t bits = (acc >> 16) - (8 - nv);       // codes < 2^12: their sum stays below bit 16
                    const uint32_t j = __umulhi(k, P.sub_magic);          // subchunk of these 8 symbols
                    atomicAdd(&sub_bits[32 * hs + j], bits);
                    uint32_t* st = reinterpret_cast<uint32_t*>(stage + hs * P.stage_stride + k + 4 * j);
                    st[0] = sy[s][0];
                    st[1] = sy[s][1];
                    ++hs;
                }
            }
        }
        __syncwarp();

        // ---- phase B: subchunk end bits, piece sizes, position of the chunk in the payload area ----
        uint32_t my_bits[2] = {0, 0}, my_end[2] = {0, 0}, piece16[2] = {0, 0};
        uint64_t tot16 = 0;
        {
            uint32_t hs = 0;
            for (int s = 0; s < 2; ++s) {
                if (P.mode[s] != ZC_MODE_HUFF) continue;
                const uint32_t b = sub_bits[32 * hs + lane];
                uint32_t inc = b;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                    if (lane >= (uint32_t)o) inc += t;
                }
                my_bits[hs] = b;
                my_end[hs] = inc;
                reinterpret_cast<uint32_t*>(P.out + P.lay.sub_end_tab[s] + 128ull * c)[lane] = inc;
                const uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, inc, 31);
                piece16[hs] = (chunk_bits + 127) / 128;
                tot16 += piece16[hs];
                if (lane == 0) atomicAdd(&P.ctl->payload_bits[s], (unsigned long long)chunk_bits);
                ++hs;
            }
        }
        uint64_t off16 = 0;
        if (n_huff) {
            if (!lookback_exclusive(P.flags, c, lane, tot16, off16)) {
                raise_status(P.ctl, ZC_E_DEVICE_TIMEOUT);
                break;
            }
        }

        // ---- phase C: each lane packs its subchunk at its final bit position ----
        {
            uint32_t hs = 0;
            uint64_t piece_off16 = off16;
            for (int s = 0; s < 2; ++s) {
                if (P.mode[s] != ZC_MODE_HUFF) continue;
                if (lane == 0) reinterpret_cast<uint32_t*>(P.out + P.lay.chunk_off_tab[s])[c] = (uint32_t)piece_off16;
                uint32_t* piece = reinterpret_cast<uint32_t*>(P.out + P.lay.payload_off + 16 * piece_off16);
                const uint32_t piece_words = 4 * piece16[hs];
                const uint32_t end = my_end[hs], start = end - my_bits[hs];
                const uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, end, 31);
                // words shared between neighbours (and the padding) start from zero and are OR-ed into
                if ((start >> 5) < piece_words) piece[start >> 5] = 0;
                if (lane == 31 && (end >> 5) < piece_words) piece[end >> 5] = 0;
                if (lane < 4 && piece_words) {
                    const uint32_t w = piece_words - 4 + lane;
                    if (32ull * w >= chunk_bits) piece[w] = 0;
                }
                __syncwarp();

                const uint32_t lo_sym = lane * P.sub;
                const uint32_t n_my = lo_sym < c_syms ? min(P.sub, c_syms - lo_sym) : 0u;
                const uint8_t* src = stage + hs * P.stage_stride + lo_sym + 4 * lane;
                const uint32_t* tab = enc + 256 * s;
                uint64_t acc = 0;
                uint32_t nb = start & 31, wi = start >> 5;
                bool first = true;
                for (uint32_t i = 0; i < n_my; i += 4) {
                    const uint32_t four = *reinterpret_cast<const uint32_t*>(src + i);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if (i + q < n_my) {
                            const uint32_t e = tab[(four >> (8 * q)) & 0xFF];
                            const uint32_t l = e >> 16;
                            acc = (acc << l) | (e & 0xFFFF);
                            nb += l;
                        }
                        if ((q & 1) && nb >= 32) {            // two codes add at most 24 bits to at most 31 pending
                            const uint32_t word = (uint32_t)(acc >> (nb - 32));
                            if (first) { atomicOr(&piece[wi], word); first = false; }
                            else piece[wi] = word;
                            ++wi;
                            nb -= 32;
                        }
                    }
                }
                if (nb >= 32) {                                // cannot happen (flushed after every pair), kept for safety
                    const uint32_t word = (uint32_t)(acc >> (nb - 32));
                    atomicOr(&piece[wi], word);
                    ++wi; nb -= 32;
                }
                if (nb && my_bits[hs]) atomicOr(&piece[wi], (uint32_t)(acc << (32 - nb)));
                piece_off16 += piece16[hs];
                ++hs;
            }
        }
        __syncwarp();

        // the warp that owns the last chunk knows the size of the whole payload area
        if (lane == 0 && c == P.n_chunks - 1) P.ctl->total16 = off16 + tot16;
    }
    if (first_bad) raise_status(P.ctl, first_bad);
}

// Writes the 128-byte header and the guard once every chunk is in place (stream order guarantees it).
__global__ void finish_kernel(const EncParams P)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const bool any_huff = P.mode[0] == ZC_MODE_HUFF || P.mode[1] == ZC_MODE_HUFF;
    const uint64_t payload_bytes = any_huff ? 16ull * P.ctl->total16 : 0;
    uint8_t* h = P.out;
    uint32_t* h32 = reinterpret_cast<uint32_t*>(h);
    unsigned long long* h64 = reinterpret_cast<unsigned long long*>(h);
    for (int i = 0; i < 32; ++i) h32[i] = 0;
    h32[0] = kMagic;
    h[kHdrVersion] = 1; h[kHdrFormat] = (uint8_t)P.format; h[kHdrStreams] = 2;
    h64[kHdrElems / 8] = P.n_elems;
    h32[kHdrChunkBytes / 4] = P.chunk_bytes;
    h32[kHdrChunks / 4] = P.n_chunks;
    h[kHdrLmax] = kLmax; h[kHdrGroup] = (uint8_t)P.group; h[kHdrSubs] = kSubs;
    const uint64_t total = P.lay.payload_off + payload_bytes + (any_huff ? 16 : 0);
    h64[kHdrTotal / 8] = total;
    h64[kHdrPayloadOff / 8] = P.lay.payload_off;
    h64[kHdrPayloadBytes / 8] = payload_bytes;
    for (int s = 0; s < 2; ++s) {
        uint8_t* d = h + kHdrStream0 + kHdrStreamStride * s;
        d[kSdMode] = (uint8_t)P.mode[s];
        reinterpret_cast<unsigned long long*>(d)[1] = P.n_syms;
        reinterpret_cast<unsigned long long*>(d)[2] = P.mode[s] == ZC_MODE_HUFF ? P.ctl->payload_bits[s] : 8 * P.n_syms;
        reinterpret_cast<unsigned long long*>(d)[3] = P.lay.section_off[s];
    }
    if (any_huff) {
        uint32_t* g = reinterpret_cast<uint32_t*>(P.out + P.lay.payload_off + payload_bytes);
        g[0] = g[1] = g[2] = g[3] = 0;
    }
    P.ctl->total16 = total;                      // the host reads the container size from here
}

// ------------------------------------------------------------------------------------------------
// decoder
// ------------------------------------------------------------------------------------------------

struct DecParams {
    const uint8_t* comp;
    uint8_t* out;
    Control* ctl;
    uint64_t comp_bytes, input_bytes, n_syms, n_elems;
    uint32_t n_chunks, cs, sub, chunk_bytes, format, group;
    uint32_t round;          // symbols each lane decodes between two cooperative merge steps
    uint32_t slot_bytes;     // per-warp staging space for compressed pieces
};

// Decode table entry: bits 7..0 bits consumed, 9..8 symbols produced (1 or 2), 15 no valid code,
// 23..16 first symbol, 31..24 second symbol.
__device__ __forceinline__ uint32_t walk_code(uint32_t window12, const uint32_t* first, const uint32_t* count,
                                              const uint32_t* offset, const uint8_t* sorted, uint32_t& len)
{
    for (uint32_t l = 1; l <= kLmax; ++l) {
        const uint32_t code = window12 >> (kLmax - l);
        const uint32_t rel = code - first[l];
        if (code >= first[l] && rel < count[l]) { len = l; return sorted[offset[l] + rel]; }
    }
    len = 0;
    return 0;
}

// Build the two-symbol decode table of one stream from its code-length table (all threads of the block).
// Returns false (to every thread) if the lengths are not a usable prefix code.
__device__ bool build_lut(const uint8_t* __restrict__ code_len, uint32_t* lut, uint32_t* scratch)
{
    // scratch: count[16] | first[16] | offset[16] | warp_count[8][16] | sorted[256 bytes] | ok
    uint32_t* count = scratch;
    uint32_t* first = scratch + 16;
    uint32_t* offset = scratch + 32;
    uint32_t* wcount = scratch + 48;                       // [8][16]
    uint8_t* sorted = reinterpret_cast<uint8_t*>(scratch + 48 + 128);
    uint32_t* ok = scratch + 48 + 128 + 64;
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid < 48 + 128) scratch[tid] = 0;
    if (tid == 0) *ok = 1;
    __syncthreads();
    uint32_t my_len = 0, my_rank = 0;
    if (tid < 256) {
        my_len = code_len[tid];
        if (my_len > kLmax) { *ok = 0; my_len = 0; }
        for (uint32_t l = 1; l <= kLmax; ++l) {
            const uint32_t m = __ballot_sync(0xFFFFFFFFu, my_len == l);
            if (my_len == l) my_rank = __popc(m & ((1u << lane) - 1));
            if (lane == 0) wcount[warp * 16 + l] = __popc(m);
        }
    }
    __syncthreads();
    if (tid == 0) {
        uint32_t code = 0, off = 0, active = 0;
        uint64_t kraft = 0;
        for (uint32_t l = 1; l <= kLmax; ++l) {
            uint32_t cnt = 0;
            for (uint32_t w = 0; w < 8; ++w) { const uint32_t t = wcount[w * 16 + l]; wcount[w * 16 + l] = cnt; cnt += t; }
            count[l] = cnt;
            code = (code + count[l - 1]) << 1;
            first[l] = code;
            offset[l] = off;
            off += cnt;
            active += cnt;
            kraft += (uint64_t)cnt << (kLmax - l);
        }
        const bool complete = kraft == (1ull << kLmax);
        const bool single = active == 1 && count[1] == 1;
        if (!(complete || single || active == 0)) *ok = 0;
    }
    __syncthreads();
    if (tid < 256 && my_len) sorted[offset[my_len] + wcount[warp * 16 + my_len] + my_rank] = (uint8_t)tid;
    __syncthreads();
    for (uint32_t idx = tid; idx < kLutEntries; idx += blockDim.x) {
        uint32_t l1, l2;
        const uint32_t s1 = walk_code(idx, first, count, offset, sorted, l1);
        uint32_t e;
        if (l1 == 0) {
            e = 0x8000u | (1u << 8) | 1u;                   // no code: keep the lane moving, flag it
        } else {
            const uint32_t rest = (idx << l1) & (kLutEntries - 1);
            const uint32_t s2 = walk_code(rest, first, count, offset, sorted, l2);
            if (l2 != 0 && l1 + l2 <= kLmax) e = (s2 << 24) | (s1 << 16) | (2u << 8) | (l1 + l2);
            else e = (s1 << 16) | (1u << 8) | l1;
        }
        lut[idx] = e;
    }
    __syncthreads();
    return *ok != 0;
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
// Bulk asynchronous copy global -> shared of this CTA, completion counted in bytes on an mbarrier.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// One lane decodes symbols of its subchunk until `target` symbols sit in its staging row.
// STAGED: the piece was copied to shared memory (pay_s is its shared address), else it is read
// from global memory.  Every table lookup yields one or two symbols; both bytes are always
// stored and the write position advances by the number that is valid.
template <bool STAGED>
__device__ __forceinline__ void decode_run(uint32_t pay_s, const uint32_t* __restrict__ pay_g, uint32_t lut_s,
                                           uint32_t row_s, uint32_t& out, uint32_t target, uint32_t& pos,
                                           uint32_t& last, uint32_t& flags)
{
    while (out < target) {
        const uint32_t w = pos >> 5;
        uint32_t hi, lo;
        if (STAGED) { hi = lds32(pay_s + 4 * w); lo = lds32(pay_s + 4 * w + 4); }
        else { hi = __ldg(pay_g + w); lo = __ldg(pay_g + w + 1); }
        uint32_t win = __funnelshift_l(lo, hi, pos);
        uint32_t e = lds32(lut_s + ((win >> (30 - kLmax)) & (4 * kLutEntries - 4)));
        sts8(row_s + out, e >> 16);
        sts8(row_s + out + 1, e >> 24);
        out += (e >> 8) & 3;
        uint32_t used = e & 0xFF;
        flags |= e;
        if (out < target) {
            win <<= used;
            e = lds32(lut_s + ((win >> (30 - kLmax)) & (4 * kLutEntries - 4)));
            sts8(row_s + out, e >> 16);
            sts8(row_s + out + 1, e >> 24);
            out += (e >> 8) & 3;
            used += e & 0xFF;
            flags |= e;
        }
        last = e;
        pos += used;
    }
}

template <int FMT>
__global__ void __launch_bounds__(512)
decode_kernel(const __grid_constant__ DecParams P)
{
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;

    // shared layout: lut[2][4096] u32 | scratch 1 KiB | per warp: mbarrier[2] | per warp: rows[2] | per warp: slot
    uint32_t* lut = reinterpret_cast<uint32_t*>(smem);
    uint32_t* scratch = lut + 2 * kLutEntries;
    uint64_t* bars = reinterpret_cast<uint64_t*>(scratch + 256);
    const uint32_t row_stride = P.round + 4;                   // bytes per lane row
    const uint32_t rows_bytes = (32 * row_stride + 15) & ~15u; // one stream's rows of a warp
    uint8_t* rows_all = reinterpret_cast<uint8_t*>(bars + 2 * n_warps);
    uint8_t* slots_all = rows_all + (size_t)n_warps * 2 * rows_bytes;
    uint8_t* rows = rows_all + (size_t)warp * 2 * rows_bytes;
    uint8_t* slot = slots_all + (size_t)warp * P.slot_bytes;
    uint64_t* bar = bars + 2 * warp;

    // ---- header check against the plan (every block does it; it is 128 bytes) ----
    __shared__ uint32_t s_mode[2];
    __shared__ uint32_t s_ok;
    __shared__ unsigned long long s_payload_off, s_payload_bytes, s_sec[2];
    if (threadIdx.x == 0) {
        const uint8_t* h = P.comp;
        const uint32_t* h32 = reinterpret_cast<const uint32_t*>(h);
        const unsigned long long* h64 = reinterpret_cast<const unsigned long long*>(h);
        bool ok = h32[0] == kMagic && h[kHdrVersion] == 1 && h[kHdrVersion + 1] == 0 && h[kHdrFormat] == P.format &&
                  h[kHdrStreams] == 2 && h64[kHdrElems / 8] == P.n_elems && h32[kHdrChunkBytes / 4] == P.chunk_bytes &&
                  h32[kHdrChunks / 4] == P.n_chunks && h[kHdrLmax] == kLmax && h[kHdrGroup] == P.group && h[kHdrSubs] == kSubs;
        uint32_t mode[2] = {0, 0};
        for (int s = 0; s < 2 && ok; ++s) {
            const uint8_t* d = h + kHdrStream0 + kHdrStreamStride * s;
            mode[s] = d[kSdMode];
            ok = mode[s] <= 1 && reinterpret_cast<const unsigned long long*>(d)[1] == P.n_syms;
        }
        if (ok) {
            // recompute where everything must be and compare with what the header says
            uint64_t off = kHeaderBytes, sec[2] = {0, 0};
            const uint64_t tab = 256 + (((uint64_t)4 * P.n_chunks + 15) & ~15ull) + 128ull * P.n_chunks;
            for (int s = 0; s < 2; ++s) if (mode[s] == ZC_MODE_HUFF) { sec[s] = off; off += tab; }
            for (int s = 0; s < 2; ++s) if (mode[s] == ZC_MODE_RAW) { sec[s] = off; off += (P.n_syms + 15) & ~15ull; }
            const bool any_huff = mode[0] == ZC_MODE_HUFF || mode[1] == ZC_MODE_HUFF;
            const uint64_t total = h64[kHdrTotal / 8], poff = h64[kHdrPayloadOff / 8], pbytes = h64[kHdrPayloadBytes / 8];
            ok = poff == off && (pbytes & 15) == 0 && total == poff + pbytes + (any_huff ? 16 : 0) && total <= P.comp_bytes;
            for (int s = 0; s < 2 && ok; ++s)
                ok = reinterpret_cast<const unsigned long long*>(h + kHdrStream0 + kHdrStreamStride * s)[3] == sec[s];
            s_mode[0] = mode[0]; s_mode[1] = mode[1];
            s_sec[0] = sec[0]; s_sec[1] = sec[1];
            s_payload_off = poff; s_payload_bytes = pbytes;
        }
        s_ok = ok ? 1u : 0u;
    }
    if (lane == 0) { mbar_init(&bar[0], 1); mbar_init(&bar[1], 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (!s_ok) { if (threadIdx.x == 0) raise_status(P.ctl, ZC_E_CORRUPT); return; }

    const bool huff0 = s_mode[0] == ZC_MODE_HUFF, huff1 = s_mode[1] == ZC_MODE_HUFF;
    const uint32_t n_huff = (huff0 ? 1u : 0u) + (huff1 ? 1u : 0u);
    bool tables_ok = true;
    if (huff0) tables_ok = build_lut(P.comp + s_sec[0], lut, scratch) && tables_ok;
    if (huff1) tables_ok = build_lut(P.comp + s_sec[1], lut + kLutEntries, scratch) && tables_ok;
    if (!tables_ok) { if (threadIdx.x == 0) raise_status(P.ctl, ZC_E_CORRUPT); return; }

    const uint64_t tab_chunk = 256, tab_sub = 256 + (((uint64_t)4 * P.n_chunks + 15) & ~15ull);
    const uint8_t* payload = P.comp + s_payload_off;
    const unsigned long long payload_bytes = s_payload_bytes;
    const uint8_t* sec0 = P.comp + s_sec[0];
    const uint8_t* sec1 = P.comp + s_sec[1];
    const uint32_t half_slot = n_huff == 2 ? (P.slot_bytes / 2) & ~15u : P.slot_bytes;
    const uint32_t R = P.round, parts = R / 8;                  // 8-symbol parts per row
    const uint32_t parts_shift = 31 - __clz(parts);             // parts is 2, 4 or 8
    uint32_t parity[2] = {0, 0};
    uint32_t err = 0;

    for (uint32_t c = blockIdx.x * n_warps + warp; c < P.n_chunks; c += gridDim.x * n_warps) {
        const uint64_t c_lo = (uint64_t)c * P.cs;
        const uint32_t c_syms = (uint32_t)min((uint64_t)P.cs, P.n_syms - c_lo);
        const uint64_t out_lo = 2 * c_lo;                       // two element bytes per symbol in every format
        const uint32_t out_bytes = (uint32_t)min((uint64_t)P.chunk_bytes, P.input_bytes - out_lo);
        const uint32_t lo_sym = lane * P.sub;
        const uint32_t n_my = lo_sym < c_syms ? min(P.sub, c_syms - lo_sym) : 0u;

        // ---- per stream: where my subchunk starts and where the chunk's piece is; check, then stage ----
        uint32_t pos[2] = {0, 0}, carry[2] = {0, 0}, carry_sym[2] = {0, 0}, piece_bytes[2] = {0, 0};
        const uint32_t* pay_g[2] = {nullptr, nullptr};
        bool staged[2] = {false, false};
        bool ok = true;
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            if (!(s == 0 ? huff0 : huff1)) continue;
            const uint8_t* sec = s == 0 ? sec0 : sec1;
            const uint32_t my_end = reinterpret_cast<const uint32_t*>(sec + tab_sub + 128ull * c)[lane];
            uint32_t start = __shfl_up_sync(0xFFFFFFFFu, my_end, 1);
            if (lane == 0) start = 0;
            const uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, my_end, 31);
            const uint32_t off16 = reinterpret_cast<const uint32_t*>(sec + tab_chunk)[c];
            piece_bytes[s] = ((chunk_bits + 127) / 128) * 16;
            ok = ok && start <= my_end && my_end <= chunk_bits && my_end - start <= n_my * kLmax &&
                 16ull * off16 + piece_bytes[s] <= payload_bytes;
            pos[s] = start;
            pay_g[s] = reinterpret_cast<const uint32_t*>(payload + 16ull * off16);
        }
        if (!__all_sync(0xFFFFFFFFu, ok)) { err = ZC_E_CORRUPT; break; }
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            if (!(s == 0 ? huff0 : huff1)) continue;
            const uint32_t hs = (s == 1 && huff0) ? 1u : 0u;
            const uint32_t copy_bytes = piece_bytes[s] + 16;    // the next piece or the guard follows: peeks stay inside
            if (copy_bytes <= half_slot) {
                staged[s] = true;
                if (lane == 0) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    mbar_expect_tx(&bar[hs], copy_bytes);
                    bulk_g2s(slot + hs * half_slot, pay_g[s], copy_bytes, &bar[hs]);
                }
            }
        }
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            if (!staged[s]) continue;
            const uint32_t hs = (s == 1 && huff0) ? 1u : 0u;
            uint32_t spins = 0;
            while (!mbar_try_wait(&bar[hs], parity[hs])) {
                if (++spins > kSpinLimit) { err = ZC_E_DEVICE_TIMEOUT; break; }
            }
            parity[hs] ^= 1;
        }
        if (__any_sync(0xFFFFFFFFu, err == ZC_E_DEVICE_TIMEOUT)) {
            // give copies in flight one more bounded chance to land before the block leaves
            for (int hs = 0; hs < 2; ++hs)
                for (uint32_t spins = 0; spins < kSpinLimit && !mbar_try_wait(&bar[hs], parity[hs] ^ 1); ++spins) {}
            err = ZC_E_DEVICE_TIMEOUT;
            break;
        }

        // ---- rounds: every lane decodes R symbols of its subchunk, then the warp merges and stores ----
        const uint32_t n_rounds = P.sub / R;
        uint32_t flags = 0;
        for (uint32_t r = 0; r < n_rounds; ++r) {
            if (r * R >= c_syms) break;                          // lane 0 has the most symbols; nothing left
            const uint32_t done = r * R;
            const uint32_t target = n_my > done ? min(R, n_my - done) : 0u;
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                if (!(s == 0 ? huff0 : huff1)) continue;
                const uint32_t hs = (s == 1 && huff0) ? 1u : 0u;
                const uint32_t row_s = smem_u32(rows + hs * rows_bytes + lane * row_stride);
                const uint32_t lut_s = smem_u32(lut + s * kLutEntries);
                uint32_t out = 0, last = 0;
                if (target) {
                    if (carry[s]) { sts8(row_s, carry_sym[s]); out = 1; }
                    if (staged[s]) decode_run<true>(smem_u32(slot + hs * half_slot), nullptr, lut_s, row_s, out, target, pos[s], last, flags);
                    else decode_run<false>(0, pay_g[s], lut_s, row_s, out, target, pos[s], last, flags);
                    carry[s] = out - target;                     // 0 or 1: a pair straddled the round boundary
                    carry_sym[s] = last >> 24;
                }
            }
            __syncwarp();
            // cooperative merge: part q covers 8 symbols = 16 output bytes
            for (uint32_t q = lane; q < 32 * parts; q += 32) {
                const uint32_t j = q >> parts_shift, p = q & (parts - 1);
                const uint32_t k = j * P.sub + r * R + p * 8;    // symbol index inside the chunk
                if (k >= c_syms) continue;
                uint32_t sy[2][2];
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    if (s == 0 ? huff0 : huff1) {
                        const uint32_t hs = (s == 1 && huff0) ? 1u : 0u;
                        const uint32_t a = smem_u32(rows + hs * rows_bytes + j * row_stride + p * 8);
                        sy[s][0] = lds32(a); sy[s][1] = lds32(a + 4);
                    } else {
                        const uint2 v = ld_nc_v2((s == 0 ? sec0 : sec1) + c_lo + k);
                        sy[s][0] = v.x; sy[s][1] = v.y;
                    }
                }
                uint32_t o[4];
                merge16<FMT>(sy[0], sy[1], o);
                const uint32_t byte = 2 * k;
                if (byte + 16 <= out_bytes) {
                    st_cs_v4(P.out + out_lo + byte, make_uint4(o[0], o[1], o[2], o[3]));
                } else {
                    for (uint32_t i = 0; byte + i < out_bytes; ++i) P.out[out_lo + byte + i] = (uint8_t)(o[i >> 2] >> (8 * (i & 3)));
                }
            }
            __syncwarp();
        }
        if (flags & 0x8000u) err = ZC_E_CORRUPT;
    }
    if (err) raise_status(P.ctl, err);
}

// ------------------------------------------------------------------------------------------------
// host side of the C ABI
// ------------------------------------------------------------------------------------------------

static int g_sm_count = 0;
static int sm_count()
{
    if (!g_sm_count) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
        g_sm_count = n;
    }
    return g_sm_count;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

constexpr size_t kMaxSmem = 227 * 1024;

}  // namespace zc

using namespace zc;

extern "C" {

zc_status zc_histogram(const zc_plan_t* p, const void* d_in, uint64_t* d_hist, void* cuda_stream)
{
    if (!p || !d_hist || (!d_in && p->n_elems) || !aligned16(d_in)) return ZC_E_INVALID_ARG;
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
        kern<<<grid, kHistThreads, smem, st>>>((const uint8_t*)d_in, p->input_bytes, p->n_syms, (unsigned long long*)d_hist);
        e = cudaGetLastError();
    };
    switch (p->format) {
    case ZC_FMT_BF16: launch(hist_kernel<ZC_FMT_BF16>); break;
    case ZC_FMT_FP8_E4M3: launch(hist_kernel<ZC_FMT_FP8_E4M3>); break;
    default: launch(hist_kernel<ZC_FMT_FP4_E2M1>); break;
    }
    return e == cudaSuccess ? ZC_OK : ZC_E_CUDA;
}

zc_status zc_compress(const zc_plan_t* p, const zc_codebook_t* cb, const void* d_in, void* d_out, size_t out_capacity,
                      void* d_workspace, uint64_t* h_out_bytes, void* cuda_stream)
{
    if (!p || !cb || !d_out || !d_workspace || (!d_in && p->n_elems)) return ZC_E_INVALID_ARG;
    if (!aligned16(d_in) || !aligned16(d_out) || !aligned16(d_workspace)) return ZC_E_INVALID_ARG;
    if (out_capacity < zc_max_compressed_bytes(p)) return ZC_E_BUFFER_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    EncParams P{};
    P.in = (const uint8_t*)d_in;
    P.out = (uint8_t*)d_out;
    P.ctl = (Control*)d_workspace;
    P.flags = (unsigned long long*)((uint8_t*)d_workspace + kControlBytes);
    P.input_bytes = p->input_bytes; P.n_syms = p->n_syms; P.n_elems = p->n_elems;
    P.n_chunks = p->n_chunks; P.cs = p->syms_per_chunk; P.sub = p->syms_per_sub; P.chunk_bytes = p->chunk_bytes;
    P.format = p->format; P.group = p->group;
    uint32_t n_huff = 0;
    for (int s = 0; s < 2; ++s) {
        // an empty tensor has no symbols to code: both streams are stored raw
        P.mode[s] = p->n_syms ? cb->mode[s] : (uint32_t)ZC_MODE_RAW;
        n_huff += P.mode[s] == ZC_MODE_HUFF;
    }
    P.lay = make_layout(*p, P.mode);
    P.stage_stride = p->syms_per_chunk + 4 * kSubs;
    P.sub_magic = (uint32_t)(((1ull << 32) + p->syms_per_sub - 1) / p->syms_per_sub);

    EncTables T;
    for (int s = 0; s < 2; ++s)
        for (int v = 0; v < 256; ++v) T.enc[s][v] = cb->len[s][v] ? ((uint32_t)cb->len[s][v] << 16) | cb->code[s][v] : 0u;

    if (cudaMemsetAsync(d_workspace, 0, kControlBytes + 8ull * p->n_chunks, st) != cudaSuccess) return ZC_E_CUDA;

    cudaError_t e = cudaSuccess;
    if (p->n_chunks) {
        const size_t fixed = 512 * sizeof(uint32_t);
        const size_t per_warp = 64 * sizeof(uint32_t) + (size_t)n_huff * P.stage_stride;
        uint32_t warps = (uint32_t)std::min<size_t>(16, (kMaxSmem - fixed - 1024) / per_warp);
        if (warps == 0) return ZC_E_UNSUPPORTED;
        const size_t smem = fixed + warps * per_warp;
        // resident blocks per SM by shared memory (leave 1 KiB per block for the system) and threads
        uint32_t per_sm = (uint32_t)std::min<size_t>(kMaxSmem / (smem + 1024), 2048 / (warps * 32));
        per_sm = std::max(per_sm, 1u);
        const uint32_t want = (p->n_chunks + warps - 1) / warps;
        const uint32_t grid = std::min<uint32_t>(want, (uint32_t)sm_count() * per_sm);
        auto launch = [&](auto kern) {
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return;
            kern<<<grid, warps * 32, smem, st>>>(P, T);
            e = cudaGetLastError();
        };
        switch (p->format) {
        case ZC_FMT_BF16: launch(encode_kernel<ZC_FMT_BF16>); break;
        case ZC_FMT_FP8_E4M3: launch(encode_kernel<ZC_FMT_FP8_E4M3>); break;
        default: launch(encode_kernel<ZC_FMT_FP4_E2M1>); break;
        }
        if (e != cudaSuccess) return ZC_E_CUDA;
    }
    finish_kernel<<<1, 32, 0, st>>>(P);
    if (cudaGetLastError() != cudaSuccess) return ZC_E_CUDA;

    if (h_out_bytes) {
        Control h;
        if (cudaMemcpyAsync(&h, d_workspace, sizeof(Control), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZC_E_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return ZC_E_CUDA;
        if (h.status) return (zc_status)h.status;
        *h_out_bytes = h.total16;
    }
    return ZC_OK;
}

zc_status zc_decompress(const zc_plan_t* p, const void* d_comp, size_t comp_bytes, void* d_out, void* d_workspace,
                        void* cuda_stream)
{
    if (!p || !d_comp || !d_workspace || (!d_out && p->n_elems)) return ZC_E_INVALID_ARG;
    if (!aligned16(d_comp) || !aligned16(d_out) || !aligned16(d_workspace)) return ZC_E_INVALID_ARG;
    if (comp_bytes < kHeaderBytes) return ZC_E_CORRUPT;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(d_workspace, 0, kControlBytes, st) != cudaSuccess) return ZC_E_CUDA;

    DecParams P{};
    P.comp = (const uint8_t*)d_comp;
    P.out = (uint8_t*)d_out;
    P.ctl = (Control*)d_workspace;
    P.comp_bytes = comp_bytes; P.input_bytes = p->input_bytes; P.n_syms = p->n_syms; P.n_elems = p->n_elems;
    P.n_chunks = p->n_chunks; P.cs = p->syms_per_chunk; P.sub = p->syms_per_sub; P.chunk_bytes = p->chunk_bytes;
    P.format = p->format; P.group = p->group;
    P.round = (p->syms_per_sub % 64 == 0) ? 64 : (p->syms_per_sub % 32 == 0) ? 32 : 16;
    P.slot_bytes = std::min<uint32_t>(p->syms_per_chunk, 16384) + 32;

    const size_t fixed = 2 * kLutEntries * sizeof(uint32_t) + 1024;
    const size_t rows_bytes = (32 * (P.round + 4) + 15) & ~15u;
    const size_t per_warp = 16 + 2 * rows_bytes + P.slot_bytes;
    uint32_t warps = (uint32_t)std::min<size_t>(16, (kMaxSmem - fixed - 2048) / per_warp);
    if (warps == 0) return ZC_E_UNSUPPORTED;
    if (warps < 8) { /* large chunks: stage less, read long pieces straight from global memory */
        P.slot_bytes = 4096 + 32;
        warps = 16;
    }
    const size_t smem = fixed + warps * (16 + 2 * rows_bytes + P.slot_bytes);
    uint32_t per_sm = (uint32_t)std::min<size_t>(kMaxSmem / (smem + 1024), 2048 / (warps * 32));
    per_sm = std::max(per_sm, 1u);
    // at least one block even for an empty tensor: the header is still checked
    const uint32_t want = std::max<uint32_t>((p->n_chunks + warps - 1) / warps, 1);
    const uint32_t grid = std::min<uint32_t>(want, (uint32_t)sm_count() * per_sm);
    cudaError_t e = cudaSuccess;
    auto launch = [&](auto kern) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return;
        kern<<<grid, warps * 32, smem, st>>>(P);
        e = cudaGetLastError();
    };
    switch (p->format) {
    case ZC_FMT_BF16: launch(decode_kernel<ZC_FMT_BF16>); break;
    case ZC_FMT_FP8_E4M3: launch(decode_kernel<ZC_FMT_FP8_E4M3>); break;
    default: launch(decode_kernel<ZC_FMT_FP4_E2M1>); break;
    }
    return e == cudaSuccess ? ZC_OK : ZC_E_CUDA;
}

zc_status zc_device_status(const zc_plan_t* p, const void* d_workspace, void* cuda_stream)
{
    if (!p || !d_workspace) return ZC_E_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint32_t status = 0;
    if (cudaMemcpyAsync(&status, d_workspace, sizeof(status), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZC_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZC_E_CUDA;
    return (zc_status)status;
}

}  // extern "C"
