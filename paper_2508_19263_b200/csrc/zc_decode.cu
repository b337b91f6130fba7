// Decoder kernel (table decode of the Huffman-coded streams fused with field merge) and zc_decompress.
//
// One warp per chunk, one lane per subchunk.  The chunk's compressed piece is staged in shared memory
// with a bulk asynchronous copy (TMA, non-multicast) completing on an mbarrier.  Work proceeds in
// rounds: every lane decodes R symbols of its own subchunk into a padded row of shared memory, then the
// whole warp merges 32 x R symbols with the other stream and writes 16-byte vectors, fully coalesced.
// Raw sign+mantissa bytes for a round are fetched into registers before the round's decoding, so the
// DRAM latency hides behind the table lookups.
#include "zc_device.cuh"

namespace zc {

struct DecParams {
    const uint8_t* comp;
    uint8_t* out;
    Control* ctl;
    uint64_t comp_bytes, input_bytes, n_syms, n_elems;
    uint32_t n_chunks, cs, sub, chunk_bytes, format, group;
    uint32_t pool_bytes;     // per-warp shared memory: symbol rows first, the rest stages compressed pieces
};

constexpr uint32_t kWideLutBytes = kLutEntries * 8;   // stream 0: up to 4 symbols per lookup
constexpr uint32_t kNarrowLutBytes = kLutEntries * 4; // stream 1: up to 2 symbols per lookup
constexpr uint32_t kScratchBytes = 1024;
constexpr uint32_t kDecFixedSmem = kWideLutBytes + kNarrowLutBytes + kScratchBytes;

__device__ __forceinline__ uint2 lds64(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts8_if(bool p, uint32_t addr, uint32_t v)
{
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\t@q st.shared.u8 [%0], %1;\n\t}"
                 :: "r"(addr), "r"(v), "r"((uint32_t)p) : "memory");
}

// ------------------------------------------------------------------------------------------------
// decode tables, built by every block from the container's code-length table
// ------------------------------------------------------------------------------------------------
// Canonical-code bookkeeping in shared memory: for each length the first code value, the number of
// codes and the offset of its symbols in the (length, symbol)-sorted list.

struct CodeBook {
    uint32_t* count;   // [16]
    uint32_t* first;   // [16]
    uint32_t* offset;  // [16]
    uint32_t* wcount;  // [8][16] per-warp counts, then exclusive prefix over warps
    uint8_t* sorted;   // [256]
    uint32_t* ok;
};

__device__ __forceinline__ CodeBook codebook_views(uint32_t* scratch)
{
    CodeBook b;
    b.count = scratch; b.first = scratch + 16; b.offset = scratch + 32; b.wcount = scratch + 48;
    b.sorted = reinterpret_cast<uint8_t*>(scratch + 48 + 128);
    b.ok = scratch + 48 + 128 + 64;
    return b;
}

// One symbol from the top bits of a 12-bit window: (len << 8) | symbol, or 0 if no code matches.
__device__ __forceinline__ uint32_t walk_code(uint32_t window12, const CodeBook& b)
{
    for (uint32_t l = 1; l <= kLmax; ++l) {
        const uint32_t code = window12 >> (kLmax - l);
        const uint32_t rel = code - b.first[l];
        if (code >= b.first[l] && rel < b.count[l]) return (l << 8) | b.sorted[b.offset[l] + rel];
    }
    return 0;
}

// Fills the table of one stream.  WIDE: 8-byte entries {symbols (up to 4, low byte first), len | cnt << 8};
// otherwise 4-byte entries len | cnt << 8 | sym1 << 16 | sym2 << 24.  `single` is a 4096 x u16 scratch table.
// Every entry yields at least one symbol, so a decoding lane always advances.  Returns false to all
// threads if the lengths are not a complete prefix code (or the one-symbol code).
template <bool WIDE>
__device__ bool build_lut(const uint8_t* __restrict__ code_len, uint8_t* lut, uint16_t* single, uint32_t* scratch)
{
    const CodeBook b = codebook_views(scratch);
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid < 48 + 128) scratch[tid] = 0;
    if (tid == 0) *b.ok = 1;
    __syncthreads();
    uint32_t my_len = 0, my_rank = 0;
    if (tid < 256) {
        my_len = code_len[tid];
        if (my_len > kLmax) { *b.ok = 0; my_len = 0; }
        for (uint32_t l = 1; l <= kLmax; ++l) {
            const uint32_t m = __ballot_sync(0xFFFFFFFFu, my_len == l);
            if (my_len == l) my_rank = __popc(m & ((1u << lane) - 1));
            if (lane == 0) b.wcount[warp * 16 + l] = __popc(m);
        }
    }
    __syncthreads();
    if (tid == 0) {
        uint32_t code = 0, off = 0, active = 0;
        uint64_t kraft = 0;
        for (uint32_t l = 1; l <= kLmax; ++l) {
            uint32_t cnt = 0;
            for (uint32_t w = 0; w < 8; ++w) { const uint32_t t = b.wcount[w * 16 + l]; b.wcount[w * 16 + l] = cnt; cnt += t; }
            b.count[l] = cnt;
            code = (code + b.count[l - 1]) << 1;
            b.first[l] = code;
            b.offset[l] = off;
            off += cnt;
            active += cnt;
            kraft += (uint64_t)cnt << (kLmax - l);
        }
        const bool complete = kraft == (1ull << kLmax);
        const bool one = active == 1 && b.count[1] == 1;
        if (!(complete || one || active == 0)) *b.ok = 0;
    }
    __syncthreads();
    if (tid < 256 && my_len) b.sorted[b.offset[my_len] + b.wcount[warp * 16 + my_len] + my_rank] = (uint8_t)tid;
    __syncthreads();
    // one symbol per window; a window no code matches (possible only for the one-symbol code) reads as
    // that list's first symbol with length 1
    for (uint32_t idx = tid; idx < kLutEntries; idx += blockDim.x) {
        uint32_t e = walk_code(idx, b);
        if (e == 0) e = (1u << 8) | b.sorted[0];
        single[idx] = (uint16_t)e;
    }
    __syncthreads();
    for (uint32_t idx = tid; idx < kLutEntries; idx += blockDim.x) {
        uint32_t rest = idx, total = 0, cnt = 0, syms = 0;
#pragma unroll
        for (int k = 0; k < (WIDE ? 4 : 2); ++k) {
            const uint32_t e = single[rest];
            const uint32_t l = e >> 8;
            if (k > 0 && total + l > kLmax) break;
            syms |= (e & 0xFF) << (8 * k);
            total += l;
            ++cnt;
            rest = (rest << l) & (kLutEntries - 1);
        }
        if (WIDE) reinterpret_cast<uint2*>(lut)[idx] = make_uint2(syms, total | (cnt << 8));
        else reinterpret_cast<uint32_t*>(lut)[idx] = total | (cnt << 8) | (syms << 16);
    }
    __syncthreads();
    return *b.ok != 0;
}

// ------------------------------------------------------------------------------------------------
// per-lane decoding of one round
// ------------------------------------------------------------------------------------------------

struct LaneStream {
    uint32_t pos;         // next bit of my subchunk, counted from the start of the chunk's piece
    uint32_t carry_n;     // symbols already decoded beyond the previous round (0..3)
    uint32_t carry_syms;  // those symbols, first one in the low byte
};

// Decode until `target` symbols sit in the lane's row.  Each pass loads a 32-bit window at the current
// bit and does two table lookups (a lookup consumes at most 12 bits); all symbol bytes of an entry are
// stored and the write position advances by the number that is valid.
template <bool WIDE, bool STAGED>
__device__ __forceinline__ void decode_round(LaneStream& st, uint32_t pay_s, const uint32_t* __restrict__ pay_g,
                                             uint32_t lut_s, uint32_t row_s, uint32_t target)
{
    uint32_t out = st.carry_n;
    if (out) sts32(row_s, st.carry_syms);
    uint32_t pos = st.pos;
    uint32_t last_syms = 0, last_meta = 0;
    while (out < target) {
        const uint32_t w = pos >> 5;
        uint32_t hi, lo;
        if (STAGED) { hi = lds32(pay_s + 4 * w); lo = lds32(pay_s + 4 * w + 4); }
        else { hi = __ldg(pay_g + w); lo = __ldg(pay_g + w + 1); }
        uint32_t win = __funnelshift_l(lo, hi, pos);
        uint32_t syms, meta;
        if (WIDE) {
            const uint2 e = lds64(lut_s + ((win >> (29 - kLmax)) & (8 * kLutEntries - 8)));
            syms = e.x; meta = e.y;
        } else {
            const uint32_t e = lds32(lut_s + ((win >> (30 - kLmax)) & (4 * kLutEntries - 4)));
            syms = e >> 16; meta = e & 0xFFFF;
        }
        const uint32_t a = row_s + out;
        sts8(a, syms); sts8(a + 1, syms >> 8);
        if (WIDE) { sts8(a + 2, syms >> 16); sts8(a + 3, syms >> 24); }
        out += meta >> 8;
        win = __funnelshift_l(0, win, meta);               // shift count = low 5 bits = bits consumed
        uint32_t used = meta;
        last_syms = syms; last_meta = meta;
        const bool more = out < target;
        {
            uint32_t syms2, meta2;
            if (WIDE) {
                const uint2 e = lds64(lut_s + ((win >> (29 - kLmax)) & (8 * kLutEntries - 8)));
                syms2 = e.x; meta2 = e.y;
            } else {
                const uint32_t e = lds32(lut_s + ((win >> (30 - kLmax)) & (4 * kLutEntries - 4)));
                syms2 = e >> 16; meta2 = e & 0xFFFF;
            }
            const uint32_t a2 = row_s + out;
            sts8_if(more, a2, syms2); sts8_if(more, a2 + 1, syms2 >> 8);
            if (WIDE) { sts8_if(more, a2 + 2, syms2 >> 16); sts8_if(more, a2 + 3, syms2 >> 24); }
            if (more) { out += meta2 >> 8; used += meta2; last_syms = syms2; last_meta = meta2; }
        }
        pos += used & 0xFF;
    }
    st.pos = pos;
    const uint32_t extra = out - target;                     // symbols of the last entry that belong to the next round
    st.carry_n = extra;
    st.carry_syms = extra ? last_syms >> (8 * ((last_meta >> 8) - extra)) : 0u;
}

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
// PPL = 16-symbol parts each lane merges per round = R / 16, R in {16, 32, 64}.

template <int FMT, int PPL>
__global__ void __launch_bounds__(1024, 1)
decode_kernel(const __grid_constant__ DecParams P)
{
    constexpr uint32_t R = 16 * PPL;
    constexpr uint32_t kRowStride = R + 4;                     // bytes; the padding spreads the lanes' rows over the banks
    constexpr uint32_t kRowsBytes = 32 * kRowStride;           // one stream's rows of a warp (multiple of 16)
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;

    uint8_t* lut0 = smem;                                      // wide table of stream 0
    uint8_t* lut1 = smem + kWideLutBytes;                      // narrow table of stream 1
    uint32_t* scratch = reinterpret_cast<uint32_t*>(smem + kWideLutBytes + kNarrowLutBytes);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kDecFixedSmem);
    uint8_t* pools = reinterpret_cast<uint8_t*>(bars + 2 * n_warps);
    uint8_t* pool = pools + (size_t)warp * P.pool_bytes;
    uint64_t* bar = bars + 2 * warp;

    // ---- header check against the plan ----
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
    {
        // the warps' pools are free until the main loop: 8 KiB of them hold the one-symbol scratch table
        uint16_t* single = reinterpret_cast<uint16_t*>(pools);
        bool tables_ok = true;
        if (huff0) tables_ok = build_lut<true>(P.comp + s_sec[0], lut0, single, scratch) && tables_ok;
        if (huff1) tables_ok = build_lut<false>(P.comp + s_sec[1], lut1, single, scratch) && tables_ok;
        if (!tables_ok) { if (threadIdx.x == 0) raise_status(P.ctl, ZC_E_CORRUPT); return; }
    }

    const uint64_t tab_chunk = 256, tab_sub = 256 + (((uint64_t)4 * P.n_chunks + 15) & ~15ull);
    const uint8_t* payload = P.comp + s_payload_off;
    const unsigned long long payload_bytes = s_payload_bytes;
    const uint8_t* sec0 = P.comp + s_sec[0];
    const uint8_t* sec1 = P.comp + s_sec[1];
    // pool: rows of stream 0 (if coded), rows of stream 1 (if coded), then one staging slot per coded stream
    const uint32_t rows0_off = 0, rows1_off = huff0 ? kRowsBytes : 0;
    const uint32_t slots_off = rows1_off + (huff1 ? kRowsBytes : 0);
    const uint32_t n_huff = (huff0 ? 1u : 0u) + (huff1 ? 1u : 0u);
    const uint32_t slot_room = P.pool_bytes > slots_off ? P.pool_bytes - slots_off : 0u;
    const uint32_t slot_bytes = n_huff ? (slot_room / n_huff) & ~15u : 0u;
    const uint32_t slot0_s = smem_u32(pool + slots_off);
    const uint32_t slot1_s = slot0_s + (huff0 ? slot_bytes : 0);
    const uint32_t rows0_s = smem_u32(pool + rows0_off), rows1_s = smem_u32(pool + rows1_off);
    const uint32_t lut0_s = smem_u32(lut0), lut1_s = smem_u32(lut1);
    const uint32_t step = gridDim.x * n_warps;
    uint32_t parity0 = 0, parity1 = 0;
    uint32_t err = 0;

    // subchunk end bits and piece offsets of the first chunk; those of the following chunk are
    // requested while the current one is decoded
    uint32_t c = blockIdx.x * n_warps + warp;
    uint32_t nx_end0 = 0, nx_off0 = 0, nx_end1 = 0, nx_off1 = 0;
    if (c < P.n_chunks) {
        if (huff0) { nx_end0 = reinterpret_cast<const uint32_t*>(sec0 + tab_sub + 128ull * c)[lane];
                     nx_off0 = reinterpret_cast<const uint32_t*>(sec0 + tab_chunk)[c]; }
        if (huff1) { nx_end1 = reinterpret_cast<const uint32_t*>(sec1 + tab_sub + 128ull * c)[lane];
                     nx_off1 = reinterpret_cast<const uint32_t*>(sec1 + tab_chunk)[c]; }
    }

    for (; c < P.n_chunks; c += step) {
        const uint64_t c_lo = (uint64_t)c * P.cs;
        const uint32_t c_syms = (uint32_t)min((uint64_t)P.cs, P.n_syms - c_lo);
        const uint64_t out_lo = 2 * c_lo;                       // two element bytes per symbol in every format
        const uint32_t out_bytes = (uint32_t)min((uint64_t)P.chunk_bytes, P.input_bytes - out_lo);
        const uint32_t lo_sym = lane * P.sub;
        const uint32_t n_my = lo_sym < c_syms ? min(P.sub, c_syms - lo_sym) : 0u;

        // ---- where my subchunk starts and where the chunk's pieces are; check, then stage ----
        LaneStream st0{0, 0, 0}, st1{0, 0, 0};
        const uint32_t* pay0_g = nullptr;
        const uint32_t* pay1_g = nullptr;
        bool staged0 = false, staged1 = false;
        uint32_t piece0 = 0, piece1 = 0;
        bool ok = true;
        if (huff0) {
            const uint32_t my_end = nx_end0, off16 = nx_off0;
            uint32_t start = __shfl_up_sync(0xFFFFFFFFu, my_end, 1);
            if (lane == 0) start = 0;
            const uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, my_end, 31);
            piece0 = ((chunk_bits + 127) / 128) * 16;
            ok = ok && start <= my_end && my_end <= chunk_bits && my_end - start <= n_my * kLmax &&
                 16ull * off16 + piece0 <= payload_bytes;
            st0.pos = start;
            pay0_g = reinterpret_cast<const uint32_t*>(payload + 16ull * off16);
        }
        if (huff1) {
            const uint32_t my_end = nx_end1, off16 = nx_off1;
            uint32_t start = __shfl_up_sync(0xFFFFFFFFu, my_end, 1);
            if (lane == 0) start = 0;
            const uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, my_end, 31);
            piece1 = ((chunk_bits + 127) / 128) * 16;
            ok = ok && start <= my_end && my_end <= chunk_bits && my_end - start <= n_my * kLmax &&
                 16ull * off16 + piece1 <= payload_bytes;
            st1.pos = start;
            pay1_g = reinterpret_cast<const uint32_t*>(payload + 16ull * off16);
        }
        if (!__all_sync(0xFFFFFFFFu, ok)) { err = ZC_E_CORRUPT; break; }
        // the copy takes 16 bytes more than the piece (the next piece or the guard), so window peeks stay inside
        if (huff0 && piece0 + 16 <= slot_bytes) {
            staged0 = true;
            if (lane == 0) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_expect_tx(&bar[0], piece0 + 16);
                bulk_g2s(pool + slots_off, pay0_g, piece0 + 16, &bar[0]);
            }
        }
        if (huff1 && piece1 + 16 <= slot_bytes) {
            staged1 = true;
            if (lane == 0) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_expect_tx(&bar[1], piece1 + 16);
                bulk_g2s(pool + slots_off + (huff0 ? slot_bytes : 0), pay1_g, piece1 + 16, &bar[1]);
            }
        }
        // request the next chunk's tables now; they are consumed in the next iteration
        {
            const uint32_t cn = c + step;
            if (cn < P.n_chunks) {
                if (huff0) { nx_end0 = reinterpret_cast<const uint32_t*>(sec0 + tab_sub + 128ull * cn)[lane];
                             nx_off0 = reinterpret_cast<const uint32_t*>(sec0 + tab_chunk)[cn]; }
                if (huff1) { nx_end1 = reinterpret_cast<const uint32_t*>(sec1 + tab_sub + 128ull * cn)[lane];
                             nx_off1 = reinterpret_cast<const uint32_t*>(sec1 + tab_chunk)[cn]; }
            }
        }

        const uint32_t n_rounds = P.sub / R;
        bool waited = false;
        for (uint32_t r = 0; r < n_rounds; ++r) {
            if (r * R >= c_syms) break;                          // lane 0 has the most symbols; nothing left
            // ---- raw stream bytes of this round go to registers before the decoding starts ----
            uint4 raw1[PPL];
#pragma unroll
            for (int i = 0; i < PPL; ++i) {
                const uint32_t q = i * 32 + lane;
                const uint32_t k = (q / PPL) * P.sub + r * R + (q % PPL) * 16;   // symbol index inside the chunk
                raw1[i] = make_uint4(0, 0, 0, 0);
                if (k < c_syms && !huff1) raw1[i] = ld_nc_v4(sec1 + c_lo + k);
            }
            if (!waited) {
                waited = true;
                if (staged0) {
                    uint32_t spins = 0;
                    while (!mbar_try_wait(&bar[0], parity0)) if (++spins > kSpinLimit) { err = ZC_E_DEVICE_TIMEOUT; break; }
                    parity0 ^= 1;
                }
                if (staged1) {
                    uint32_t spins = 0;
                    while (!mbar_try_wait(&bar[1], parity1)) if (++spins > kSpinLimit) { err = ZC_E_DEVICE_TIMEOUT; break; }
                    parity1 ^= 1;
                }
                if (__any_sync(0xFFFFFFFFu, err == ZC_E_DEVICE_TIMEOUT)) { err = ZC_E_DEVICE_TIMEOUT; break; }
            }
            // ---- every lane decodes R symbols of its subchunk ----
            const uint32_t done = r * R;
            const uint32_t target = n_my > done ? min(R, n_my - done) : 0u;
            if (target) {
                if (huff0) {
                    const uint32_t row_s = rows0_s + lane * kRowStride;
                    if (staged0) decode_round<true, true>(st0, slot0_s, nullptr, lut0_s, row_s, target);
                    else decode_round<true, false>(st0, 0, pay0_g, lut0_s, row_s, target);
                }
                if (huff1) {
                    const uint32_t row_s = rows1_s + lane * kRowStride;
                    if (staged1) decode_round<false, true>(st1, slot1_s, nullptr, lut1_s, row_s, target);
                    else decode_round<false, false>(st1, 0, pay1_g, lut1_s, row_s, target);
                }
            }
            __syncwarp();
            // ---- cooperative merge: part q covers 16 symbols = 32 output bytes ----
#pragma unroll
            for (int i = 0; i < PPL; ++i) {
                const uint32_t q = i * 32 + lane;
                const uint32_t j = q / PPL, p = q % PPL;
                const uint32_t k = j * P.sub + r * R + p * 16;
                if (k >= c_syms) continue;
                uint32_t e[4], s[4];
                if (huff0) {
                    const uint32_t a = rows0_s + j * kRowStride + p * 16;
                    e[0] = lds32(a); e[1] = lds32(a + 4); e[2] = lds32(a + 8); e[3] = lds32(a + 12);
                } else {
                    const uint4 v = ld_nc_v4(sec0 + c_lo + k);
                    e[0] = v.x; e[1] = v.y; e[2] = v.z; e[3] = v.w;
                }
                if (huff1) {
                    const uint32_t a = rows1_s + j * kRowStride + p * 16;
                    s[0] = lds32(a); s[1] = lds32(a + 4); s[2] = lds32(a + 8); s[3] = lds32(a + 12);
                } else { s[0] = raw1[i].x; s[1] = raw1[i].y; s[2] = raw1[i].z; s[3] = raw1[i].w; }
                uint32_t o[8];
                merge16<FMT>(e, s, o);
                merge16<FMT>(e + 2, s + 2, o + 4);
                const uint32_t byte = 2 * k;
                uint8_t* dst = P.out + out_lo + byte;
                if (byte + 32 <= out_bytes) {
                    st_cs_v4(dst, make_uint4(o[0], o[1], o[2], o[3]));
                    st_cs_v4(dst + 16, make_uint4(o[4], o[5], o[6], o[7]));
                } else {
#pragma unroll
                    for (int t = 0; t < 32; ++t)
                        if (byte + t < out_bytes) dst[t] = (uint8_t)(o[t >> 2] >> (8 * (t & 3)));
                }
            }
            __syncwarp();
        }
        if (err) break;
    }
    if (__any_sync(0xFFFFFFFFu, err == ZC_E_DEVICE_TIMEOUT)) {
        // give copies in flight one more bounded chance to land before the block leaves
        for (uint32_t spins = 0; spins < kSpinLimit && !mbar_try_wait(&bar[0], parity0 ^ 1); ++spins) {}
        for (uint32_t spins = 0; spins < kSpinLimit && !mbar_try_wait(&bar[1], parity1 ^ 1); ++spins) {}
    }
    if (err) raise_status(P.ctl, err);
}

}  // namespace zc

using namespace zc;

extern "C" {

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

    // symbols per round and lane: the largest of 64 / 32 / 16 that divides the subchunk length
    const uint32_t ppl = (p->syms_per_sub % 64 == 0) ? 4 : (p->syms_per_sub % 32 == 0) ? 2 : 1;
    const uint32_t rows_bytes = 32 * (16 * ppl + 4);
    // per warp: one stream's rows plus room to stage a piece as large as the raw chunk stream; pieces that
    // do not fit (or chunks above 16 KiB of symbols) are read from global memory instead
    P.pool_bytes = std::max<uint32_t>(rows_bytes + std::min<uint32_t>(p->syms_per_chunk, 16384) + 32, 2 * rows_bytes);
    const size_t fixed = kDecFixedSmem + 64 /* static shared */;
    size_t per_warp = 16 + P.pool_bytes;
    uint32_t warps = (uint32_t)std::min<size_t>(32, (kMaxSmem - fixed - 1024) / per_warp);
    if (warps < 8) {                 // large chunks: stage less
        P.pool_bytes = std::max<uint32_t>(rows_bytes + 4096 + 32, 2 * rows_bytes);
        per_warp = 16 + P.pool_bytes;
        warps = (uint32_t)std::min<size_t>(32, (kMaxSmem - fixed - 1024) / per_warp);
    }
    // the table build uses 8 KiB of the pools and 256 threads
    while (warps * (size_t)P.pool_bytes < 8192) ++warps;
    if (warps < 8 || warps > 32) return ZC_E_UNSUPPORTED;
    const size_t smem = kDecFixedSmem + warps * per_warp;
    // at least one block even for an empty tensor: the header is still checked
    const uint32_t want = std::max<uint32_t>((p->n_chunks + warps - 1) / warps, 1);
    const uint32_t grid = std::min<uint32_t>(want, (uint32_t)sm_count());
    cudaError_t e = cudaSuccess;
    auto launch = [&](auto kern) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return;
        kern<<<grid, warps * 32, smem, st>>>(P);
        e = cudaGetLastError();
    };
#define ZC_DEC_CASE(F)                                                     \
    if (ppl == 4) launch(decode_kernel<F, 4>);                             \
    else if (ppl == 2) launch(decode_kernel<F, 2>);                        \
    else launch(decode_kernel<F, 1>);
    switch (p->format) {
    case ZC_FMT_BF16: ZC_DEC_CASE(ZC_FMT_BF16) break;
    case ZC_FMT_FP8_E4M3: ZC_DEC_CASE(ZC_FMT_FP8_E4M3) break;
    default: ZC_DEC_CASE(ZC_FMT_FP4_E2M1) break;
    }
#undef ZC_DEC_CASE
    return e == cudaSuccess ? ZC_OK : ZC_E_CUDA;
}

}  // extern "C"
