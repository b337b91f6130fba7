// Encoder kernels (split, code-length scan, bit packing) and zc_compress / zc_device_status.
#include "zc_device.cuh"

namespace zc {

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

}  // namespace zc

using namespace zc;

extern "C" {

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
