// Encoder kernels (split, code-length scan, bit packing) and zc_compress / zc_device_status.
#include "zc_device.cuh"

namespace zc {

// ------------------------------------------------------------------------------------------------
// encoder
// ------------------------------------------------------------------------------------------------

// Per symbol: the code left-aligned in bits 31..20 and its length in bits 3..0; a symbol without a code is 16.
struct EncTables { uint32_t enc[2][256]; };

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
    uint32_t stage_stride;                       // bytes of one coded stream's lane regions per warp
    uint32_t region_bytes;                       // one lane region: (n_slots + 1) * sub + 4
    uint32_t sub_width;                          // bytes per sub_end entry (2 or 4)
    uint32_t n_slots;                            // pack slots per lane region (1..3, see encode_kernel)
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

// Per-warp shared memory of one coded stream: 32 lane regions (+4 bytes of padding each, which also makes
// the region stride an odd number of words so that lanes walking their regions hit different banks).
// A region is cut into slots of `sub` bytes: n_slots pack slots followed by the symbols,
//   [pack 0 | .. | pack n_slots-1 | symbols].
// A lane packs the codes of its subchunk into pack slot (batch index mod n_slots), so the packed bits of the
// last n_slots batches are alive at the same time and the copy-out of a batch can wait up to n_slots
// iterations for the batch's position in the payload area (which comes from a look-back over other blocks).
// Packing into the last slot may run on into the symbols behind it: codes are at most 12 bits, so after k
// symbols at most 1.5 k bytes are written while the read position is sub + k, and the writer never passes
// unread symbols.  Packing into any other slot stops at the slot's end.  The packed bits of a subchunk
// normally fit one slot (8 bits per symbol); a chunk in which some lane needs more is finished on a slow
// path (everything older is copied out, then the chunk is packed again from slot 0 with the whole region
// as room) before anything else is staged.

__device__ __forceinline__ void sts32_if(bool p, uint32_t addr, uint32_t v)
{
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\t@q st.shared.u32 [%0], %1;\n\t}"
                 :: "r"(addr), "r"(v), "r"((uint32_t)p) : "memory");
}

// Append `len` bits (given left-aligned in `code`, zero below them) to a lane's bit accumulator and write a
// full 32-bit word to the region when one is complete and lies below `limit`.  hi holds the nb (< 32)
// pending bits left-aligned.
__device__ __forceinline__ void put_bits(uint32_t code, uint32_t len, uint32_t& hi, uint32_t& nb, uint32_t& waddr, uint32_t limit)
{
    hi |= code >> nb;
    const uint32_t lo = __funnelshift_r(0, code, nb);           // the bits that do not fit: code << (32 - nb), 0 if nb == 0
    const uint32_t n = nb + len;
    const bool full = n >= 32;
    sts32_if(full && waddr < limit, waddr, hi);
    waddr += full ? 4 : 0;
    hi = full ? lo : hi;
    nb = n & 31;
}

__device__ __forceinline__ unsigned long long ld_ctl(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// Writes the 128-byte header and the guard; called by one thread once every chunk is in place.
__device__ void write_header(const EncParams& P)
{
    const bool any_huff = P.mode[0] == ZC_MODE_HUFF || P.mode[1] == ZC_MODE_HUFF;
    const uint64_t payload_bytes = any_huff ? 16ull * ld_ctl(&P.ctl->total16) : 0;
    uint8_t* h = P.out;
    uint32_t* h32 = reinterpret_cast<uint32_t*>(h);
    unsigned long long* h64 = reinterpret_cast<unsigned long long*>(h);
    for (int i = 0; i < 32; ++i) h32[i] = 0;
    h32[0] = kMagic;
    h[kHdrVersion] = 1; h[kHdrFormat] = (uint8_t)P.format; h[kHdrStreams] = 2;
    h64[kHdrElems / 8] = P.n_elems;
    h32[kHdrChunkBytes / 4] = P.chunk_bytes;
    h32[kHdrChunks / 4] = P.n_chunks;
    h[kHdrLmax] = kLmax; h[kHdrGroup] = (uint8_t)P.group; h[kHdrSubs] = kSubs; h[kHdrSubWidth] = (uint8_t)P.sub_width;
    const uint64_t total = P.lay.payload_off + payload_bytes + (any_huff ? 16 : 0);
    h64[kHdrTotal / 8] = total;
    h64[kHdrPayloadOff / 8] = P.lay.payload_off;
    h64[kHdrPayloadBytes / 8] = payload_bytes;
    for (int s = 0; s < 2; ++s) {
        uint8_t* d = h + kHdrStream0 + kHdrStreamStride * s;
        d[kSdMode] = (uint8_t)P.mode[s];
        reinterpret_cast<unsigned long long*>(d)[1] = P.n_syms;
        reinterpret_cast<unsigned long long*>(d)[2] = P.mode[s] == ZC_MODE_HUFF ? ld_ctl(&P.ctl->payload_bits[s]) : 8 * P.n_syms;
        reinterpret_cast<unsigned long long*>(d)[3] = P.lay.section_off[s];
    }
    if (any_huff) {
        uint32_t* g = reinterpret_cast<uint32_t*>(P.out + P.lay.payload_off + payload_bytes);
        g[0] = g[1] = g[2] = g[3] = 0;
    }
    P.ctl->total16 = total;                      // the host reads the container size from here
}


// For an empty tensor no encoder block runs: the header is all there is.
__global__ void finish_kernel(const EncParams P)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) write_header(P);
}

constexpr uint32_t kEncMaxWorkers = 8;       // worker warps per block = chunks per batch; one more warp does the look-back

// What a worker warp keeps about a chunk between packing it and copying it out.
struct PackedChunk {
    uint32_t c;                 // chunk index; kNoChunk: this warp had no chunk in the batch
    uint32_t end[2];            // per stream: inclusive scan of the subchunks' bit counts over the lanes (= sub_end)
};
constexpr uint32_t kNoChunk = 0xFFFFFFFFu;

template <int FMT>
__global__ void __launch_bounds__((kEncMaxWorkers + 1) * 32, 3)
encode_kernel(const __grid_constant__ EncParams P, const __grid_constant__ EncTables T)
{
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n_workers = (blockDim.x >> 5) - 1;
    const bool scanner = warp == n_workers;                     // the last warp only does the look-back
    const bool huff0 = P.mode[0] == ZC_MODE_HUFF, huff1 = P.mode[1] == ZC_MODE_HUFF;
    const uint32_t n_huff = (huff0 ? 1u : 0u) + (huff1 ? 1u : 0u);
    const uint32_t n_slots = P.n_slots;

    // shared: enc[2][256] | per worker warp: regions[n_huff][stage_stride]
    uint32_t* enc = reinterpret_cast<uint32_t*>(smem);
    uint8_t* stage_all = smem + 2048;
    for (uint32_t i = threadIdx.x; i < 512; i += blockDim.x) enc[i] = T.enc[i >> 8][i & 255];
    uint8_t* stage = stage_all + (size_t)(scanner ? 0 : warp) * n_huff * P.stage_stride;
    const uint32_t region = P.region_bytes;                     // (n_slots + 1) * sub + 4
    const uint32_t sym_off = n_slots * P.sub;                   // symbols sit at this offset inside a region

    // The warps of a block are coupled only through these words (no block barrier inside the loop):
    //   s_base[it & 3], s_base_seq   first chunk of the block's batch `it`; seq = batches handed out so far
    //   s_tot[it & 3][w], s_cnt[..]  payload size of worker w's chunk; cnt = workers that have posted it
    //   s_off[it & 3][w], s_off_seq  position of that chunk in the payload area; seq = batches placed so far
    // A worker has consumed the position of batch `it - n_slots` (n_slots <= 3) before it posts a size for
    // batch `it`, and the look-back warp places a batch only after every worker has posted, so no warp is more
    // than three batches away from any other and four copies of each word are enough.
    __shared__ uint32_t s_base[4], s_base_seq, s_cnt[4], s_off_seq, s_fail;
    __shared__ unsigned long long s_tot[4][kEncMaxWorkers], s_off[4][kEncMaxWorkers];

    // block 0 writes the static parts of the table sections and the tail padding of raw bodies
    if (blockIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            if (P.mode[s] == ZC_MODE_HUFF) {
                for (uint32_t v = threadIdx.x; v < 256; v += blockDim.x) P.out[P.lay.section_off[s] + v] = (uint8_t)(T.enc[s][v] & 15);
                const uint32_t padded = (P.n_chunks + 3) & ~3u;
                for (uint32_t i = P.n_chunks + threadIdx.x; i < padded; i += blockDim.x)
                    reinterpret_cast<uint32_t*>(P.out + P.lay.chunk_off_tab[s])[i] = 0;
            } else {
                const uint64_t lo = (P.n_syms + 7) & ~7ull, hi = (P.n_syms + 15) & ~15ull;
                for (uint64_t i = lo + threadIdx.x; i < hi; i += blockDim.x) P.out[P.lay.section_off[s] + i] = 0;
            }
        }
    }
    if (threadIdx.x == 0) {
        s_fail = 0; s_cnt[0] = 0; s_cnt[1] = 0; s_cnt[2] = 0; s_cnt[3] = 0; s_off_seq = 0;
        s_base[0] = atomicAdd(&P.ctl->ticket, n_workers);       // batches of n_workers consecutive chunks
        s_base_seq = 1;
    }
    __syncthreads();

    // Bounded wait of a whole warp until a sequence word reaches `target`; false on a failure flag or when
    // the wait gives up (the caller then raises the failure flag itself).
    auto wait_seq = [&](const uint32_t* word, const uint32_t target) -> bool {
        bool ok = false;
        for (uint32_t n = 0; n < kSpinLimit; ++n) {
            if (*reinterpret_cast<const volatile uint32_t*>(word) >= target) { ok = true; break; }
            if (*reinterpret_cast<const volatile uint32_t*>(&s_fail)) break;
            if (n > 64) __nanosleep(40);
        }
        __syncwarp();
        __threadfence_block();
        return ok;
    };

    // ---- copy-out of a packed chunk: every lane moves its bits to their final position in the piece ----
    auto copy_out = [&](const PackedChunk& pc, const uint32_t slot, const uint64_t off16) {
        uint32_t hs = 0;
        uint64_t piece_off16 = off16;
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            if (P.mode[s] != ZC_MODE_HUFF) continue;
            const uint32_t end = pc.end[s];
            uint32_t start = __shfl_up_sync(0xFFFFFFFFu, end, 1);
            if (lane == 0) start = 0;
            const uint32_t bits = end - start;
            const uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, end, 31);
            const uint32_t piece16 = (chunk_bits + 127) / 128;
            if (lane == 0) reinterpret_cast<uint32_t*>(P.out + P.lay.chunk_off_tab[s])[pc.c] = (uint32_t)piece_off16;
            uint32_t* piece = reinterpret_cast<uint32_t*>(P.out + P.lay.payload_off + 16 * piece_off16);
            const uint32_t piece_words = 4 * piece16;
            const uint32_t reg_s = smem_u32(stage + hs * P.stage_stride + lane * region) + slot;
            const uint32_t sh = start & 31, d0 = start >> 5;
            const uint32_t n_dst = (sh + bits + 31) / 32;             // destination words I touch
            const uint32_t n_src = (bits + 31) / 32;
            if (__all_sync(0xFFFFFFFFu, bits >= 32)) {
                // every lane spans a word boundary, so a destination word is shared by at most two neighbouring
                // lanes: a lane hands its ragged last word to the next lane, which merges it into its first word
                const bool ragged = ((sh + bits) & 31) != 0;
                const uint32_t il = n_dst - 1;
                const uint32_t lc = il < n_src ? lds32(reg_s + 4 * il) : 0u;
                const uint32_t lp = il >= 1 ? lds32(reg_s + 4 * (il - 1)) : 0u;
                const uint32_t tail = ragged ? __funnelshift_r(lc, lp, sh) : 0u;
                uint32_t head = __shfl_up_sync(0xFFFFFFFFu, tail, 1);
                if (lane == 0) head = 0;
                const uint32_t n_mine = n_dst - ((ragged && lane != 31) ? 1u : 0u);
                uint32_t prev = 0;
                for (uint32_t i = 0; i < n_mine; ++i) {
                    const uint32_t cur = i < n_src ? lds32(reg_s + 4 * i) : 0u;
                    uint32_t v = __funnelshift_r(cur, prev, sh);      // (prev:cur) >> sh, low word
                    prev = cur;
                    if (i == 0) v |= head;
                    piece[d0 + i] = v;
                }
                if (lane < 4 && piece_words) {                        // zero padding up to the 16-byte boundary
                    const uint32_t w = piece_words - 4 + lane;
                    if (32ull * w >= chunk_bits) piece[w] = 0;
                }
            } else {
                // general case (short or empty subchunks): words shared between neighbours (and the padding)
                // start from zero and are OR-ed into
                if ((start >> 5) < piece_words) piece[start >> 5] = 0;
                if (lane == 31 && (end >> 5) < piece_words) piece[end >> 5] = 0;
                if (lane < 4 && piece_words) {
                    const uint32_t w = piece_words - 4 + lane;
                    if (32ull * w >= chunk_bits) piece[w] = 0;
                }
                __syncwarp();
                if (bits) {
                    uint32_t prev = 0;
                    for (uint32_t i = 0; i < n_dst; ++i) {
                        const uint32_t cur = i < n_src ? lds32(reg_s + 4 * i) : 0u;
                        const uint32_t v = __funnelshift_r(cur, prev, sh);
                        prev = cur;
                        // the first word may hold the previous lane's bits, a ragged last word the next lane's
                        const bool shared_word = i == 0 || (i == n_dst - 1 && ((sh + bits) & 31) != 0);
                        if (shared_word) atomicOr(&piece[d0 + i], v);
                        else piece[d0 + i] = v;
                    }
                }
            }
            piece_off16 += piece16;
            ++hs;
        }
        // the warp that owns the last chunk knows the size of the whole payload area
        if (lane == 0 && pc.c == P.n_chunks - 1) P.ctl->total16 = piece_off16;
        __syncwarp();
    };

    uint32_t bad = 0;

    if (scanner) {
        // ---- the look-back warp places batch after batch; the workers are a batch ahead of it ----
        for (uint32_t it = 0; n_huff; ++it) {
            if (!wait_seq(&s_base_seq, it + 1)) { s_fail = 1; break; }
            const uint32_t base = *reinterpret_cast<const volatile uint32_t*>(&s_base[it & 3]);
            if (base >= P.n_chunks) break;
            bool ok = false;
            for (uint32_t n = 0; n < kSpinLimit; ++n) {             // every worker posts a size (0 without a chunk)
                if (*reinterpret_cast<const volatile uint32_t*>(&s_cnt[it & 3]) == n_workers) { ok = true; break; }
                if (*reinterpret_cast<const volatile uint32_t*>(&s_fail)) break;
                __nanosleep(40);
            }
            __syncwarp();
            __threadfence_block();
            if (!ok) { s_fail = 1; break; }
            if (lane == 0) s_cnt[it & 3] = 0;
            unsigned long long v = lane < n_workers ? *reinterpret_cast<const volatile unsigned long long*>(&s_tot[it & 3][lane]) : 0ull, inc = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                if (lane >= (uint32_t)o) inc += t;
            }
            const unsigned long long batch_total = __shfl_sync(0xFFFFFFFFu, inc, 31);
            uint64_t batch_off = 0;
            ok = lookback_exclusive(P.flags, base / n_workers, lane, batch_total, batch_off);
            if (lane < n_workers) s_off[it & 3][lane] = batch_off + inc - v;
            __threadfence_block();
            __syncwarp();
            if (!ok) { s_fail = 1; break; }
            if (lane == 0) *reinterpret_cast<volatile uint32_t*>(&s_off_seq) = it + 1;
        }
    } else {
    // packed chunks that wait for their copy-out, newest first: q0 is batch it - 1, q1 batch it - 2, ...
    PackedChunk q0{kNoChunk, {0, 0}}, q1 = q0, q2 = q0;
    uint32_t n_pend = 0;
    uint32_t slot_idx = 0;                                      // pack slot of batch `it`: it mod n_slots
    // waits until the oldest pending batch is placed and copies this warp's chunk of it out
    auto flush_oldest = [&](const uint32_t it) -> bool {
        const uint32_t j = it - n_pend;                         // the batch in question
        if (n_huff) {
            if (!wait_seq(&s_off_seq, j + 1)) return false;
            PackedChunk pc;
            pc.c = n_pend == 1 ? q0.c : n_pend == 2 ? q1.c : q2.c;
            pc.end[0] = n_pend == 1 ? q0.end[0] : n_pend == 2 ? q1.end[0] : q2.end[0];
            pc.end[1] = n_pend == 1 ? q0.end[1] : n_pend == 2 ? q1.end[1] : q2.end[1];
            // its slot: the slots are used round-robin, so it lies n_pend steps behind the current one
            const uint32_t sl = (slot_idx + n_slots * 4 - n_pend) % n_slots;
            if (pc.c != kNoChunk) copy_out(pc, sl * P.sub, *reinterpret_cast<const volatile unsigned long long*>(&s_off[j & 3][warp]));
        }
        --n_pend;
        return true;
    };
    bool failed = false;
    for (uint32_t it = 0;; ++it) {
        if (!wait_seq(&s_base_seq, it + 1)) { failed = true; break; }
        const uint32_t base = *reinterpret_cast<const volatile uint32_t*>(&s_base[it & 3]);
        const bool have = base < P.n_chunks;
        if (!have) {
            while (n_pend && !failed) failed = !flush_oldest(it);
            break;
        }

        const bool active = base + warp < P.n_chunks;
        PackedChunk cur{active ? base + warp : kNoChunk, {0, 0}};
        const uint32_t slot = slot_idx * P.sub;
        const uint64_t c_lo = (uint64_t)(active ? cur.c : 0) * P.cs;
        const uint32_t c_syms = active ? (uint32_t)min((uint64_t)P.cs, P.n_syms - c_lo) : 0u;

        // ---- phase A: coalesced load, split, raw stream stored as is, coded stream staged per subchunk ----
        auto stage_group = [&](const uint4 x, const uint32_t k) {
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
            uint32_t sy[2][2];
            split16<FMT>(w, sy[0], sy[1]);
            uint32_t hs = 0;
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                if (P.mode[s] == ZC_MODE_RAW) {
                    st_cs_v2(P.out + P.lay.section_off[s] + c_lo + k, make_uint2(sy[s][0], sy[s][1]));
                } else {
                    const uint32_t j = __umulhi(k, P.sub_magic);          // subchunk of these 8 symbols
                    uint32_t* st = reinterpret_cast<uint32_t*>(stage + hs * P.stage_stride + j * region + sym_off + (k - j * P.sub));
                    st[0] = sy[s][0];
                    st[1] = sy[s][1];
                    ++hs;
                }
            }
        };
        const uint32_t n_vec = (c_syms + 7) / 8;
        const uint8_t* src_c = P.in + 2 * c_lo;
        uint32_t g = lane;
        if (2 * (c_lo + 8ull * n_vec) <= P.input_bytes) {           // every group of this chunk is complete
            for (; g + 96 < n_vec; g += 128) {                          // four loads in flight per lane
                const uint4 x0 = ld_nc_v4(src_c + 16 * g);
                const uint4 x1 = ld_nc_v4(src_c + 16 * (g + 32));
                const uint4 x2 = ld_nc_v4(src_c + 16 * (g + 64));
                const uint4 x3 = ld_nc_v4(src_c + 16 * (g + 96));
                stage_group(x0, 8 * g);
                stage_group(x1, 8 * (g + 32));
                stage_group(x2, 8 * (g + 64));
                stage_group(x3, 8 * (g + 96));
            }
            for (; g < n_vec; g += 32) stage_group(ld_nc_v4(src_c + 16 * g), 8 * g);
        } else {
            for (; g < n_vec; g += 32) stage_group(load16_guarded(P.in, 2 * (c_lo + 8ull * g), P.input_bytes), 8 * g);
        }
        __syncwarp();

        // the chunk that was packed into this slot n_slots batches ago must leave before this one is packed
        if (n_pend == n_slots && !flush_oldest(it)) { failed = true; break; }

        // ---- phase B: every lane packs the codes of its subchunk into its pack slot, from bit 0 ----
        const uint32_t lo_sym = lane * P.sub;
        const uint32_t n_my = lo_sym < c_syms ? min(P.sub, c_syms - lo_sym) : 0u;
        // returns the bit count; stores stop at `room` bytes (the count goes on)
        auto pack = [&](const int s, const uint32_t hs, const uint32_t slot, const uint32_t room) -> uint32_t {
            const uint32_t reg_s = smem_u32(stage + hs * P.stage_stride + lane * region);
            const uint32_t tab_s = smem_u32(enc + 256 * s);
            const uint32_t w0 = reg_s + slot, limit = w0 + room;
            uint32_t hi = 0, nb = 0, waddr = w0, seen = 0;
            const uint32_t src = reg_s + sym_off;
            const uint32_t full_words = n_my / 4;
            for (uint32_t i = 0; i < full_words; ++i) {
                const uint32_t four = lds32(src + 4 * i);
                const uint32_t e0 = lds32(tab_s + ((four << 2) & 0x3FC));
                const uint32_t e1 = lds32(tab_s + ((four >> 6) & 0x3FC));
                const uint32_t e2 = lds32(tab_s + ((four >> 14) & 0x3FC));
                const uint32_t e3 = lds32(tab_s + ((four >> 22) & 0x3FC));
                seen |= e0 | e1 | e2 | e3;
                // two codes at a time: the second one shifted behind the first (shift count = low 5 bits of the
                // first entry = its length); the length fields end up below bit 8 and are masked off
                const uint32_t ca = (e0 | (e1 >> (e0 & 31))) & 0xFFFFFF00u;
                put_bits(ca, (e0 + e1) & 31, hi, nb, waddr, limit);
                const uint32_t cb = (e2 | (e3 >> (e2 & 31))) & 0xFFFFFF00u;
                put_bits(cb, (e2 + e3) & 31, hi, nb, waddr, limit);
            }
            for (uint32_t i = 4 * full_words; i < n_my; ++i) {      // ragged end of the last chunk
                const uint32_t four = lds32(src + (i & ~3u));
                const uint32_t e = lds32(tab_s + (((four >> (8 * (i & 3))) & 0xFF) << 2));
                seen |= e;
                put_bits(e & 0xFFFFFF00u, e & 31, hi, nb, waddr, limit);
            }
            if (active && waddr < limit) sts32(waddr, hi);          // pending bits (or zero)
            bad |= seen & 16;                                       // an entry without a code carries bit 4
            return 8 * (waddr - w0) + nb;
        };
        bool oversize = false;
        uint32_t my_bits[2] = {0, 0};
        const bool last_slot = slot_idx + 1 == n_slots;
        {
            uint32_t hs = 0;
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                if (P.mode[s] != ZC_MODE_HUFF) continue;
                // anything beyond a slot other than the last one would overwrite an older chunk in the next slot
                my_bits[s] = pack(s, hs, slot, last_slot ? 2 * P.sub : P.sub);
                // more than 8 bits per symbol: the bits beyond the slot do not survive the next staging
                oversize |= my_bits[s] > 8 * P.sub;
                ++hs;
            }
        }

        // the ticket of the next batch is taken as late as possible (batches must start in the order they
        // were handed out, or the look-back of other blocks waits for a batch that is not even begun); its
        // latency hides behind phase C
        uint32_t next_base = 0;
        if (threadIdx.x == 0) next_base = atomicAdd(&P.ctl->ticket, n_workers);

        // ---- phase C: subchunk end bits and the chunk's size in the payload area ----
        uint64_t tot16 = 0;
        {
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                if (P.mode[s] != ZC_MODE_HUFF) continue;
                uint32_t inc = my_bits[s];
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                    if (lane >= (uint32_t)o) inc += t;
                }
                cur.end[s] = inc;
                if (active) {
                    if (P.sub_width == 2) reinterpret_cast<uint16_t*>(P.out + P.lay.sub_end_tab[s] + 64ull * cur.c)[lane] = (uint16_t)inc;
                    else reinterpret_cast<uint32_t*>(P.out + P.lay.sub_end_tab[s] + 128ull * cur.c)[lane] = inc;
                    const uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, inc, 31);
                    tot16 += (chunk_bits + 127) / 128;
                    if (lane == 0) atomicAdd(&P.ctl->payload_bits[s], (unsigned long long)chunk_bits);
                }
            }
        }
        if (lane == 0 && n_huff) {
            s_tot[it & 3][warp] = tot16;
            __threadfence_block();
            atomicAdd(&s_cnt[it & 3], 1u);
        }
        if (threadIdx.x == 0) {
            s_base[(it + 1) & 3] = next_base;
            __threadfence_block();
            *reinterpret_cast<volatile uint32_t*>(&s_base_seq) = it + 2;
        }

        q2 = q1; q1 = q0; q0 = cur;
        ++n_pend;
        slot_idx = last_slot ? 0 : slot_idx + 1;
        if (__any_sync(0xFFFFFFFFu, oversize)) {
            // some subchunk needs more than 8 bits per symbol: finish this chunk before anything else is staged.
            // Once everything older has left, a packing that was clipped at the end of its slot is redone from
            // slot 0 with the rest of the region as room.
            while (n_pend > 1 && !failed) failed = !flush_oldest(it + 1);
            if (failed) break;
            if (!last_slot) {
                uint32_t hs = 0;
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    if (P.mode[s] != ZC_MODE_HUFF) continue;
                    pack(s, hs, 0, 2 * P.sub);
                    ++hs;
                }
                __syncwarp();
                slot_idx = 1;                                   // the chunk now sits in slot 0, one behind
            }
            if (!flush_oldest(it + 1)) { failed = true; break; }
            slot_idx = 0;                                       // nothing is pending: start over with slot 0
        }
    }
    if (failed) s_fail = 1;
    }
    if (s_fail && threadIdx.x == 0) raise_status(P.ctl, 0, ZC_E_DEVICE_TIMEOUT);
    if (bad) raise_status(P.ctl, 0, ZC_E_NO_CODE);
    // the block that finishes last writes the header (every block's results are fenced before its count)
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(&P.ctl->done, 1u) == gridDim.x - 1) {
            __threadfence();
            write_header(P);
        }
    }
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
    // as many pack slots per lane region (up to 3) as still leave three blocks of 8 worker warps per SM
    P.n_slots = 1;
    for (uint32_t ns = 3; ns > 1; --ns) {
        const size_t block = 2048 + (size_t)kEncMaxWorkers * std::max<uint32_t>(n_huff, 1) * kSubs * ((ns + 1) * p->syms_per_sub + 4);
        if (3 * (block + 1024) <= kMaxSmem + 1024) { P.n_slots = ns; break; }
    }
    P.region_bytes = (P.n_slots + 1) * p->syms_per_sub + 4;
    P.sub_width = sub_end_width(p->chunk_bytes);
    P.stage_stride = kSubs * P.region_bytes;
    P.sub_magic = (uint32_t)(((1ull << 32) + p->syms_per_sub - 1) / p->syms_per_sub);

    EncTables T;
    for (int s = 0; s < 2; ++s)
        for (int v = 0; v < 256; ++v)
            T.enc[s][v] = cb->len[s][v] ? (cb->code[s][v] << (32 - cb->len[s][v])) | cb->len[s][v] : 16u;

    if (cudaMemsetAsync(d_workspace, 0, kControlBytes + 8ull * p->n_chunks, st) != cudaSuccess) return ZC_E_CUDA;

    cudaError_t e = cudaSuccess;
    if (p->n_chunks) {
        const size_t fixed = 512 * sizeof(uint32_t);
        const size_t per_warp = std::max<size_t>((size_t)n_huff * P.stage_stride, 16);
        // blocks of up to 8 worker warps (a batch of 8 consecutive chunks) plus the look-back warp; several
        // blocks per SM so that loading, packing and copy-out phases of different blocks overlap
        const uint32_t workers = (uint32_t)std::min<size_t>(kEncMaxWorkers, (kMaxSmem - fixed - 1024) / per_warp);
        if (workers == 0) return ZC_E_UNSUPPORTED;
        const uint32_t warps = workers + 1;
        const size_t smem = fixed + workers * per_warp;
        uint32_t per_sm = (uint32_t)std::min<size_t>((kMaxSmem + 1024) / (smem + 1024 + 1024), 3);
        per_sm = std::max(per_sm, 1u);
        const uint32_t want = (p->n_chunks + workers - 1) / workers;
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
    if (p->n_chunks == 0) {
        finish_kernel<<<1, 32, 0, st>>>(P);
        if (cudaGetLastError() != cudaSuccess) return ZC_E_CUDA;
    }

    if (h_out_bytes) {
        Control h;
        if (cudaMemcpyAsync(&h, d_workspace, sizeof(Control), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZC_E_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return ZC_E_CUDA;
        if (h.status & 0xFF) return (zc_status)(h.status & 0xFF);
        *h_out_bytes = h.total16;
    }
    return ZC_OK;
}

// ---- compression without a caller-supplied workspace ---------------------------------------------
// The scratch zc_compress needs (control block + one look-back word per chunk) for up to
// ZC_NOALLOC_MAX_CHUNKS chunks, resident in every GPU that loads the library.  Host code must not pass
// this symbol to a kernel: on the host its name is only a stand-in, the device address comes from
// cudaGetSymbolAddress and differs per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[ZC_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_noalloc_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device; looked up once per device.
zc_status noalloc_scratch(void** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ZC_E_CUDA;
    if (!g_noalloc_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return ZC_E_CUDA;
        g_noalloc_ptr[dev] = ptr;
    }
    *out = g_noalloc_ptr[dev];
    return ZC_OK;
}
}  // namespace

zc_status zc_compress_noalloc(const zc_plan_t* p, const zc_codebook_t* cb, const void* d_in, void* d_out,
                              size_t out_capacity, uint64_t* h_out_bytes, void* cuda_stream)
{
    if (!p) return ZC_E_INVALID_ARG;
    if (p->n_chunks > ZC_NOALLOC_MAX_CHUNKS || zc_workspace_bytes(p) > ZC_NOALLOC_SCRATCH_BYTES) return ZC_E_TOO_LARGE;
    void* scratch = nullptr;
    const zc_status st = noalloc_scratch(&scratch);
    if (st != ZC_OK) return st;
    // zc_compress clears the control block and the look-back words it uses before launching
    return zc_compress(p, cb, d_in, d_out, out_capacity, scratch, h_out_bytes, cuda_stream);
}

zc_status zc_device_status(const zc_plan_t* p, const void* d_workspace, void* cuda_stream)
{
    if (!p || !d_workspace) return ZC_E_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    unsigned long long word[2] = {0, 0};            // status, call id
    if (cudaMemcpyAsync(word, d_workspace, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZC_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZC_E_CUDA;
    // an error word left by an earlier call carries that call's id and does not count
    return (word[0] >> 8) == word[1] ? (zc_status)(word[0] & 0xFF) : ZC_OK;
}

}  // extern "C"
