// Decoder kernel (table decode of the Huffman-coded streams fused with field merge) and zc_decompress.
//
// One warp per chunk, one lane per subchunk.  The chunk's compressed piece is staged in shared memory
// with a bulk asynchronous copy (TMA, non-multicast) completing on an mbarrier.  Work proceeds in
// rounds: every lane decodes R symbols of its own subchunk into a padded row of shared memory, then the
// whole warp merges 32 x R symbols with the other stream and writes 16-byte vectors, fully coalesced.
// Raw sign+mantissa bytes for a round are fetched into registers before the round's decoding, so the
// DRAM latency hides behind the table lookups.
#include "zc_device.cuh"

#include <atomic>
#include <chrono>

namespace zc {

struct DecParams {
    const uint8_t* comp;
    const uint8_t* base;     // XOR-delta form: the decoded tensor is XOR-ed with this one before it is written; or null
    uint8_t* out;
    Control* ctl;
    uint64_t comp_bytes, input_bytes, n_syms, n_elems;
    uint32_t n_chunks, cs, sub, chunk_bytes, format, group;
    uint32_t pool_bytes;     // per-warp shared memory: symbol rows first, the rest stages compressed pieces
    uint32_t c_begin, c_end; // chunks the launch decodes (zc_decompress: all of them)
    uint32_t spec;           // the container is long enough to read stream 0's tables before the header is checked
    uint32_t spin_limit;     // polls after which a wait for a staged piece gives up
    uint32_t skip_copy;      // test hook: the copies of the pieces are not started
    uint32_t sliced;         // large chunks: pieces are staged slice by slice and lane by lane (see run_chunks)
    unsigned long long call_id;
};

// One tensor of a batch, and the parameters of a batched launch.  The tensors share format and chunk size;
// the chunks of all of them form one index space that is cut into equal contiguous ranges, one per block.
struct DecItem {
    const uint8_t* comp;
    const uint8_t* base;
    uint8_t* out;
    uint64_t comp_bytes, input_bytes, n_syms, n_elems;
    uint32_t n_chunks, first_chunk;          // first_chunk = chunks of all earlier tensors of the launch
};
constexpr uint32_t kDecBatchMax = 448;       // tensors per launch: the parameter block stays below 32 KiB
struct DecBatchParams {
    Control* ctl;
    unsigned long long call_id;
    uint32_t cs, sub, chunk_bytes, format, group, pool_bytes;
    uint32_t n_tensors, total_chunks, tensor_base, n_ranges;
    uint32_t spin_limit, skip_copy, sliced;
    DecItem item[kDecBatchMax];
};

constexpr uint32_t kLutBytes = kLutEntries * 4;       // one decode table: 4096 entries of 4 bytes
constexpr uint32_t kScratchBytes = 1280;           // code bookkeeping of build_lut (258 words)
constexpr uint32_t kDecMaxWarps = 28;              // 896 threads: 72 registers per thread fit the register file
// Launches that expect both streams to be coded (scale bytes, deltas) keep two bit readers per lane going and stage two
// pieces per warp: fewer warps fit the shared memory anyway, and the kernels built for them get more registers.
constexpr uint32_t kDecMaxWarpsBoth = 20;          // 640 threads: 96 registers per thread
template <int FMT, bool XOR>
constexpr uint32_t dec_block_warps() { return (XOR || FMT == ZC_FMT_SCALE_U8) ? kDecMaxWarpsBoth : kDecMaxWarps; }
constexpr uint32_t kDecFixedSmem = 2 * kLutBytes + kScratchBytes;
constexpr uint32_t kSliceSyms = 128;               // symbols a lane decodes from one slice of its subchunk
constexpr uint32_t kSliceBytes = 256;              // copied per slice: 15 bytes of alignment + 128 * 12 bits + the window's look-ahead fit
constexpr uint32_t kSliceSlot = 272;               // a lane's slot

__device__ __forceinline__ void sts32_if(bool p, uint32_t addr, uint32_t v)
{
    if (p) ZC_DBG_SHARED(addr, 4, return);
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\t@q st.shared.u32 [%0], %1;\n\t}"
                 :: "r"(addr), "r"(v), "r"((uint32_t)p) : "memory");
}
__device__ __forceinline__ uint32_t lds32_if(bool p, uint32_t addr)
{
    if (p) ZC_DBG_SHARED(addr, 4, return 0);
    uint32_t v;
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\tmov.u32 %0, 0;\n\t@q ld.shared.u32 %0, [%1];\n\t}"
                 : "=r"(v) : "r"(addr), "r"((uint32_t)p));
    return v;
}

// ------------------------------------------------------------------------------------------------
// decode tables, built by every block from the container's code-length table
// ------------------------------------------------------------------------------------------------
// Canonical-code bookkeeping in shared memory, per code length l = 1..12:
//   count[l]  codes of that length            first[l]  value of the first one
//   offset[l] position of its symbols in the (length, symbol)-sorted list
//   limit[l]  windows below this value start with a code of length <= l
struct CodeBook {
    uint32_t* count;   // [16]
    uint32_t* first;   // [16]
    uint32_t* offset;  // [16]
    uint32_t* limit;   // [16]
    uint32_t* wcount;  // [8][16] per-warp counts, then exclusive prefix over warps
    uint8_t* sorted;   // [256]
    uint32_t* ok;      // [0] lengths usable, [1] symbols per lookup
};

__device__ __forceinline__ CodeBook codebook_views(uint32_t* scratch)
{
    CodeBook b;
    b.count = scratch; b.first = scratch + 16; b.offset = scratch + 32; b.limit = scratch + 48; b.wcount = scratch + 64;
    b.sorted = reinterpret_cast<uint8_t*>(scratch + 64 + 128);
    b.ok = scratch + 64 + 128 + 64;
    return b;
}

// Fills the table of one stream and decides how many symbols every lookup yields (returned in *per_lookup).
//   two-symbol mode   entry bits  7..0  bits the lookup consumes      15..8 first symbol     23..16 second symbol
//                                27..24 length of the first code       31   "only the first symbol is valid"
//   one-symbol mode   entry bits  7..0  length of the code              31..24 the symbol
// Two-symbol mode: a lookup normally yields the two symbols whose codes start the 12-bit window; when the two
// codes together are longer than 12 bits the entry carries the first one and bit 31, and the decoder fetches
// the second with one more lookup.  That mode is chosen when such pairs are rare (estimated from the code
// lengths with p(symbol) = 2^-length, an eighth of that for the two longest lengths); otherwise every lookup
// yields exactly one symbol.  A fixed number of
// symbols per lookup lets a lane assemble words of 4 symbols in registers without any bookkeeping.
// `single` is a 4096 x u16 scratch table (length << 8 | symbol of the first code of every window).
// Returns false to all threads if the lengths are not a complete prefix code (or the one-symbol code).
static __device__ bool build_lut(uint32_t my_len, uint32_t* lut, uint16_t* single, uint32_t* scratch, uint32_t* per_lookup)
{
    const CodeBook b = codebook_views(scratch);
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t my_rank = 0;                                        // my_len: length of symbol tid's code (threads < 256)
    if (tid < 64 + 128) scratch[tid] = 0;
    if (tid == 0) b.ok[0] = 1;
    __syncthreads();
    if (tid < 256) {
        if (my_len > kLmax) { b.ok[0] = 0; my_len = 0; }
        for (uint32_t l = 1; l <= kLmax; ++l) {
            const uint32_t m = __ballot_sync(0xFFFFFFFFu, my_len == l);
            if (my_len == l) my_rank = __popc(m & ((1u << lane) - 1));
            if (lane == 0) b.wcount[warp * 16 + l] = __popc(m);
        }
    }
    __syncthreads();
    if (tid >= 1 && tid <= kLmax) {                              // thread l adds up length l over the 8 warps
        uint32_t cnt = 0;
        for (uint32_t w = 0; w < 8; ++w) { const uint32_t t = b.wcount[w * 16 + tid]; b.wcount[w * 16 + tid] = cnt; cnt += t; }
        b.count[tid] = cnt;
    }
    __syncthreads();
    if (tid == 0) {
        uint32_t code = 0, off = 0, active = 0;
        uint32_t p[kLmax + 2];                                    // weight of length l in units of 2^-12
        for (uint32_t l = 1; l <= kLmax; ++l) {
            const uint32_t cnt = b.count[l];
            code = (code + b.count[l - 1]) << 1;
            b.first[l] = code;
            b.offset[l] = off;
            b.limit[l] = (code + cnt) << (kLmax - l);
            off += cnt;
            active += cnt;
            p[l] = cnt << (kLmax - l);
            // codes at or next to the length limit belong to symbols that are rarer than 2^-length says: the limit
            // clipped them, or they are the never-seen symbols of a static dictionary
            if (l + 1 >= kLmax) p[l] >>= 3;
        }
        const bool complete = b.limit[kLmax] == kLutEntries;      // Kraft sum is exactly one
        const bool one = active == 1 && b.count[1] == 1;
        if (!(complete || one || active == 0)) b.ok[0] = 0;
        // probability (units of 2^-24) that two consecutive codes need more than 12 bits
        uint64_t long_pairs = 0;
        uint32_t tail = 0;                                        // sum of p[l2] for l2 >= 13 - l1
        for (uint32_t l1 = 1; l1 <= kLmax; ++l1) {
            tail += p[kLmax + 1 - l1];
            long_pairs += (uint64_t)p[l1] * tail;
        }
        b.ok[1] = long_pairs <= (1ull << 24) / 32 ? 2u : 1u;
        if (one) b.limit[1] = kLutEntries;                        // the unused half of the windows reads as the one symbol
    }
    __syncthreads();
    const uint32_t mode = b.ok[1];
    if (tid < 256 && my_len) b.sorted[b.offset[my_len] + b.wcount[warp * 16 + my_len] + my_rank] = (uint8_t)tid;
    uint32_t lim[kLmax + 1];
#pragma unroll
    for (uint32_t l = 1; l <= kLmax; ++l) lim[l] = b.limit[l];
    __syncthreads();
    // first code of every window: its length is the number of limits at or below the window value, plus one
    for (uint32_t idx = tid; idx < kLutEntries; idx += blockDim.x) {
        uint32_t l = 1;
#pragma unroll
        for (uint32_t k = 1; k < kLmax; ++k) l += idx >= lim[k] ? 1u : 0u;
        uint32_t rel = (idx >> (kLmax - l)) - b.first[l];
        if (rel >= b.count[l]) rel = 0;                           // only reachable with damaged or one-symbol tables
        single[idx] = (uint16_t)((l << 8) | b.sorted[b.offset[l] + rel]);
    }
    __syncthreads();
    for (uint32_t idx = tid; idx < kLutEntries; idx += blockDim.x) {
        const uint32_t e1 = single[idx];
        const uint32_t l1 = e1 >> 8, s1 = e1 & 0xFF;
        uint32_t e = l1 | (s1 << 24);                             // one-symbol mode: length | symbol << 24
        if (mode == 2) {
            e = l1 | (s1 << 8) | (l1 << 24);
            const uint32_t e2 = single[(idx << l1) & (kLutEntries - 1)];
            const uint32_t l2 = e2 >> 8, s2 = e2 & 0xFF;
            if (l1 + l2 <= kLmax) e = (l1 + l2) | (s1 << 8) | (s2 << 16) | (l1 << 24);
            else e |= 0x80000000u;
        }
        lut[idx] = e;
    }
    __syncthreads();
    if (tid == 0) *per_lookup = mode;
    return b.ok[0] != 0;
}

// ------------------------------------------------------------------------------------------------
// per-lane decoding of one round
// ------------------------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t load_sub_end(const uint8_t* tab, uint32_t width, uint32_t chunk, uint32_t lane)
{
    if (width == 2) return reinterpret_cast<const uint16_t*>(tab + 64ull * chunk)[lane];
    return reinterpret_cast<const uint32_t*>(tab + 128ull * chunk)[lane];
}

// A lane's place in its chunk's piece is one number, the bit position `pos`.  Piece staged in shared memory: pos
// counts from shared address 0 (8 * byte address of the slot + bit in the piece), so a window costs a shift, a mask,
// two loads and a funnel shift, and nothing else has to be kept between lookups (no pointer, no count of valid
// bits, no second buffer word).  Piece read from global memory: pos counts from the start of the piece and the
// word index is clamped to `lim`, the last place from which two words can be read.
// Bounds of the staged form: a lane starts inside its piece (checked against the tables before the chunk is
// decoded) and consumes at most 12 bits per symbol, so it reads less than 1.5 * sub + 16 bytes past the piece
// whatever the payload bits are; the block's shared memory ends with that much slack behind the last warp's
// slot.  With a valid container a lane reads at most 16 bytes past its piece (covered by the copy); with a
// damaged payload it decodes garbage in bounds and the consumed-bits check after the chunk reports the damage.

// The two payload words a lane's windows come from, kept in registers between lookups: w0, w1 = the aligned
// words that hold bits [32 i, 32 i + 64) of shared memory, next = 32 (i + 1), with i = pos / 32.  A lane consumes at
// most 24 bits between two windows, so pos crosses at most one word boundary: then w1 moves to w0 and one word
// is loaded (a predicated load in which only the lanes that crossed take part: about one word per 32 bits of
// payload instead of two words per window).
#define ZC_LANE_BITS uint32_t &pos, uint32_t &w0, uint32_t &w1, uint32_t &next
#define ZC_LANE_ARGS pos, w0, w1, next

__device__ __forceinline__ void lane_start(ZC_LANE_BITS, uint32_t at)
{
    ZC_DBG_SHARED((at >> 3) & ~3u, 4, return); ZC_DBG_SHARED(((at >> 3) & ~3u) + 4, 4, return);
    const uint32_t a = (at >> 3) & ~3u;
    pos = at;
    asm volatile("ld.shared.u32 %0, [%2];\n\tld.shared.u32 %1, [%2+4];" : "=r"(w0), "=r"(w1) : "r"(a));
    next = (at & ~31u) + 32;
}
__device__ __forceinline__ uint32_t window_s(ZC_LANE_BITS)
{
    const bool cross = pos >= next;
    const uint32_t w2 = lds32_if(cross, (next >> 3) + 4);
    w0 = cross ? w1 : w0;
    w1 = cross ? w2 : w1;
    next += cross ? 32u : 0u;
    return __funnelshift_l(w1, w0, pos);                        // the shift takes the low 5 bits of pos
}
__device__ __forceinline__ uint32_t window_g(const uint32_t* __restrict__ pay, uint32_t pos, uint32_t lim)
{
    const uint32_t w = min(pos >> 5, lim);
    return __funnelshift_l(__ldg(pay + w + 1), __ldg(pay + w), pos);
}
__device__ __forceinline__ uint32_t lut_peek(uint32_t win, uint32_t lut_s)
{
    return lds32(lut_s + 4u * (win >> (32 - kLmax)));           // window = top 12 bits; scaled by the address add
}
// pos + low byte of x, in one multiply-add-like instruction off the integer ALU pipe
__device__ __forceinline__ uint32_t add_low_byte(uint32_t pos, uint32_t x) { return __dp4a(x, 1u, pos); }

__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    ZC_DBG_SHARED(addr, 16, return);
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" :: "r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    ZC_DBG_SHARED(addr, 16, return make_uint4(0, 0, 0, 0));
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// Decode one word of 4 symbols from a piece staged in shared memory.  K = symbols per lookup (1 or 2).
// A window of 32 bits serves two lookups of at most 12 bits each.
// Two-symbol mode: entry = bits | first symbol << 8 | second symbol << 16 | first length << 24 | flag << 31.  A
// lookup whose second code did not fit the window carries the flag (rare by construction of the mode) and
// consumes its first code only, so the two lookups still end on a code boundary, one symbol short (two if both
// carry the flag); the missing symbols come from a fresh window.
// One-symbol mode: entry = length | symbol << 24, so that `pos += entry` advances the position and leaves the
// symbol in bits the position does not use.
template <int K>
__device__ __forceinline__ uint32_t decode_word(ZC_LANE_BITS, uint32_t lut_s)
{
    uint32_t win = window_s(ZC_LANE_ARGS);
    if (K == 2) {
        const uint32_t e0 = lut_peek(win, lut_s);
        const uint32_t e1 = lut_peek(__funnelshift_l(0, win, e0), lut_s);   // consume: low 5 bits of the entry
        pos = add_low_byte(pos, e0 + e1);                    // the sum of two bit counts stays below 256
        if ((int)(e0 | e1) < 0) {
            win = window_s(ZC_LANE_ARGS);
            const uint32_t f = lut_peek(win, lut_s), lf = (f >> 24) & 15;
            pos += lf;
            if ((int)(e0 & e1) < 0) {                            // both: first symbols of e0, e1, f and of one more lookup
                const uint32_t g = lut_peek(__funnelshift_l(0, win, lf), lut_s);
                pos += (g >> 24) & 15;
                return __byte_perm(__byte_perm(e0, e1, 0x0051), __byte_perm(f, g, 0x0051), 0x5410);
            }
            // e0 short: e0's first, e1's two; e1 short: e0's two, e1's first; then f's first
            return __byte_perm(__byte_perm(e0, e1, (int)e0 < 0 ? 0x0651 : 0x0521), f, 0x5210);
        }
        return __byte_perm(e0, e1, 0x6521);
    }
    const uint32_t a = lut_peek(win, lut_s);
    const uint32_t bb = lut_peek(__funnelshift_l(0, win, a), lut_s);
    pos = add_low_byte(pos, a + bb);
    win = window_s(ZC_LANE_ARGS);
    const uint32_t c = lut_peek(win, lut_s);
    const uint32_t d = lut_peek(__funnelshift_l(0, win, c), lut_s);
    pos = add_low_byte(pos, c + d);
    return __byte_perm(__byte_perm(a, bb, 0x0073), __byte_perm(c, d, 0x0073), 0x5410);
}

// Decoded symbols of a round, per coded stream and warp: lane L owns PPL quads (16 symbols = 16 bytes each);
// its quad q lives in 16-byte slot L * PPL + (q ^ f(L)), f(L) = (L >> (3 - log2 PPL)) & (PPL - 1).  With this
// placement both the writers (32 lanes, same q, one 16-byte store each) and the readers of the merge (lane l
// reads quad l % PPL of row l / PPL + i * 32 / PPL) touch eight different 16-byte bank groups per quarter warp:
// no bank conflicts on either side, one store per 16 symbols and one load per merged part.
template <int K, int PPL, bool FULL>
__device__ __forceinline__ void decode_round(ZC_LANE_BITS, uint32_t lut_s, uint32_t wr_s, uint32_t fw, uint32_t n_quads)
{
#pragma unroll
    for (int q = 0; q < PPL; ++q) {
        if (!FULL && (uint32_t)q >= n_quads) break;
        const uint32_t s0 = decode_word<K>(ZC_LANE_ARGS, lut_s);
        const uint32_t s1 = decode_word<K>(ZC_LANE_ARGS, lut_s);
        const uint32_t s2 = decode_word<K>(ZC_LANE_ARGS, lut_s);
        const uint32_t s3 = decode_word<K>(ZC_LANE_ARGS, lut_s);
        sts128(wr_s + 16 * ((uint32_t)q ^ fw), s0, s1, s2, s3);
    }
}

// Two coded streams: the same words, decoded for both streams side by side.  A lane's two bit readers are independent
// chains of dependent operations (window -> lookup -> shift -> lookup); issued alternately, one chain's shared-memory
// latency is covered by the other's arithmetic.  word_first makes the window and the two lookups that every word
// needs; word_second finishes the word: two more lookups from a second window in one-symbol mode, the rare extra
// lookups of short pair entries in two-symbol mode.  Together they compute exactly what decode_word computes.
template <int K>
__device__ __forceinline__ void word_first(ZC_LANE_BITS, uint32_t lut_s, uint32_t& x, uint32_t& y)
{
    const uint32_t win = window_s(ZC_LANE_ARGS);
    x = lut_peek(win, lut_s);
    y = lut_peek(__funnelshift_l(0, win, x), lut_s);
    pos = add_low_byte(pos, x + y);
}
template <int K>
__device__ __forceinline__ uint32_t word_second(ZC_LANE_BITS, uint32_t lut_s, const uint32_t e0, const uint32_t e1)
{
    if (K == 2) {
        if ((int)(e0 | e1) < 0) {
            const uint32_t win = window_s(ZC_LANE_ARGS);
            const uint32_t f = lut_peek(win, lut_s), lf = (f >> 24) & 15;
            pos += lf;
            if ((int)(e0 & e1) < 0) {
                const uint32_t g = lut_peek(__funnelshift_l(0, win, lf), lut_s);
                pos += (g >> 24) & 15;
                return __byte_perm(__byte_perm(e0, e1, 0x0051), __byte_perm(f, g, 0x0051), 0x5410);
            }
            return __byte_perm(__byte_perm(e0, e1, (int)e0 < 0 ? 0x0651 : 0x0521), f, 0x5210);
        }
        return __byte_perm(e0, e1, 0x6521);
    }
    const uint32_t win = window_s(ZC_LANE_ARGS);
    const uint32_t c = lut_peek(win, lut_s);
    const uint32_t d = lut_peek(__funnelshift_l(0, win, c), lut_s);
    pos = add_low_byte(pos, c + d);
    return __byte_perm(__byte_perm(e0, e1, 0x0073), __byte_perm(c, d, 0x0073), 0x5410);
}
template <int K0, int K1, int PPL, bool FULL>
__device__ __forceinline__ void decode_round2(uint32_t& posa, uint32_t& wa0, uint32_t& wa1, uint32_t& nexta, uint32_t luta_s, uint32_t wra_s,
                                              uint32_t& posb, uint32_t& wb0, uint32_t& wb1, uint32_t& nextb, uint32_t lutb_s, uint32_t wrb_s,
                                              uint32_t fw, uint32_t n_quads)
{
#pragma unroll
    for (int q = 0; q < PPL; ++q) {
        if (!FULL && (uint32_t)q >= n_quads) break;
        uint32_t a[4], b[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t ax, ay, bx, by;
            word_first<K0>(posa, wa0, wa1, nexta, luta_s, ax, ay);
            word_first<K1>(posb, wb0, wb1, nextb, lutb_s, bx, by);
            a[j] = word_second<K0>(posa, wa0, wa1, nexta, luta_s, ax, ay);
            b[j] = word_second<K1>(posb, wb0, wb1, nextb, lutb_s, bx, by);
        }
        sts128(wra_s + 16 * ((uint32_t)q ^ fw), a[0], a[1], a[2], a[3]);
        sts128(wrb_s + 16 * ((uint32_t)q ^ fw), b[0], b[1], b[2], b[3]);
    }
}

// A chunk without payload bits holds nothing but the stream's fill symbol, the symbol with the all-zero code:
// the first symbol of the table entry for a window of zeros.
static __device__ __noinline__ void fill_quads(uint32_t lut_s, uint32_t pairs, uint32_t wr_s, uint32_t fw, uint32_t n_quads)
{
    const uint32_t e = lds32(lut_s);
    const uint32_t word = (pairs ? (e >> 8) & 0xFFu : e >> 24) * 0x01010101u;
    for (uint32_t q = 0; q < n_quads; ++q) sts128(wr_s + 16 * (q ^ fw), word, word, word, word);
}

// The same result as decode_round one symbol at a time, from the first code of every table entry (two-symbol
// tables: symbol in bits 15..8, length in bits 27..24; one-symbol tables: symbol in bits 31..24, length in bits
// 3..0), reading the piece from global memory.  Small and slow on purpose: it serves pieces that were too long
// to stage.  Returns the new position.
static __device__ __noinline__ uint32_t decode_quads_global(uint32_t pos, const uint32_t* __restrict__ pay, uint32_t lut_s, uint32_t pairs,
                                                     uint32_t wr_s, uint32_t fw, uint32_t n_quads, uint32_t lim)
{
    for (uint32_t i = 0; i < 4 * n_quads; ++i) {
        uint32_t word = 0, win = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if ((k & 1) == 0) win = window_g(pay, pos, lim);
            const uint32_t e = lut_peek(win, lut_s);
            const uint32_t l = pairs ? (e >> 24) & 15 : e & 15, sy = pairs ? (e >> 8) & 0xFF : e >> 24;
            win = __funnelshift_l(0, win, l);
            pos += l;
            word |= sy << (8 * k);
        }
        sts32(wr_s + 16 * ((i >> 2) ^ fw) + 4 * (i & 3), word);
    }
    return pos;
}

// ------------------------------------------------------------------------------------------------
// chunk loop of one warp, specialised for which streams are Huffman-coded
// ------------------------------------------------------------------------------------------------

struct DecShared {                   // what the block's prologue leaves for the chunk loop
    uint32_t lut0_s, lut1_s;         // shared addresses of the decode tables
    uint32_t pairs0, pairs1;         // the stream's table yields two symbols per lookup
    unsigned long long sec0, sec1;   // byte offsets of the streams' sections
    unsigned long long payload_off, payload_bytes;
    uint32_t pool_bytes;             // bytes of this warp's pool
};

template <bool V> struct BoolTag { static constexpr bool value = V; };

// PPL = 16-symbol parts each lane merges per round = R / 16, R in {16, 32, 64}.
template <int FMT, int PPL, bool H0, bool H1, bool XOR>
__device__ __forceinline__ uint32_t run_chunks(const DecParams& P, const DecShared& S, uint8_t* pool, uint64_t* bar,
                                               uint32_t first_end0, uint32_t first_off0,
                                               uint32_t c, const uint32_t c_end, const uint32_t step,
                                               uint32_t& parity0, uint32_t& parity1)
{
    constexpr uint32_t R = 16 * PPL;
    constexpr uint32_t kLog = PPL == 4 ? 2 : PPL == 2 ? 1 : 0;
    constexpr uint32_t kRowsBytes = 512 * PPL;                 // one stream's decoded symbols of a warp and round
    constexpr uint32_t kHuff = (H0 ? 1u : 0u) + (H1 ? 1u : 0u);
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t sub_w = P.chunk_bytes <= 8192 ? 2u : 4u;
    const uint64_t tab_chunk = 256, tab_sub = 256 + (((uint64_t)4 * P.n_chunks + 15) & ~15ull);
    const uint8_t* sec0 = P.comp + S.sec0;
    const uint8_t* sec1 = P.comp + S.sec1;
    const uint8_t* payload = P.comp + S.payload_off;
    const uint64_t payload16 = S.payload_bytes >> 4;

    // pool: symbols of stream 0 (if coded), of stream 1 (if coded), then one staging slot per coded stream
    constexpr uint32_t rows1_off = H0 ? kRowsBytes : 0;
    constexpr uint32_t slots_off = rows1_off + (H1 ? kRowsBytes : 0);
    const uint32_t slot_room = S.pool_bytes > slots_off ? S.pool_bytes - slots_off : 0u;
    const uint32_t slot_bytes = kHuff ? (slot_room / (kHuff ? kHuff : 1)) & ~15u : 0u;
    const uint32_t rows0_s = smem_u32(pool), rows1_s = rows0_s + rows1_off;
    // A piece that does not fit its slot is staged in slices instead, lane by lane (where the geometry allows:
    // subchunks of a multiple of kSliceSyms symbols, slots of at least 32 lane slots): the stream's slot becomes 32
    // lane slots of kSliceSlot bytes, and every kSliceSyms symbols each lane copies the next kSliceBytes of its own
    // subchunk there.  The copy is waited for on the spot, so this is slower than staging the piece as a whole,
    // and much faster than decoding it from global memory.
    const bool can_slice = P.sliced && slot_bytes >= 32 * kSliceSlot;
    const uint32_t base0_s = rows0_s + slots_off, base1_s = base0_s + (H0 ? slot_bytes : 0u);
    uint32_t slot0_s = base0_s, slot1_s = base1_s;
    bool sliced0 = false, sliced1 = false;
    constexpr uint32_t kRoundsPerSlice = kSliceSyms / R;
    // where this lane writes its quads and reads the parts it merges (see decode_round)
    const uint32_t fw = (lane >> (3 - kLog)) & (PPL - 1);
    const uint32_t wr_off = 16 * PPL * lane;
    const uint32_t rl = lane / PPL, rq = lane % PPL;
    const uint32_t rd_off = 16 * (rl * PPL + (rq ^ ((rl >> (3 - kLog)) & (PPL - 1))));   // part i: + 512 * i
    uint32_t err = 0;

    // this lane's parts of a round: part i covers symbols k_lane + i * k_step (+ round offset) of the chunk
    const uint32_t k_lane = rl * P.sub + rq * 16, k_step = (32 / PPL) * P.sub;
    const uint32_t n_rounds = P.sub / R;
    // every chunk but possibly the last one is complete
    const uint32_t n_full = ((uint64_t)P.n_chunks * P.cs == P.n_syms && (uint64_t)P.n_chunks * P.chunk_bytes == P.input_bytes)
                                ? P.n_chunks : P.n_chunks - 1;

    uint32_t nx_end0 = first_end0, nx_off0 = first_off0, nx_end1 = 0, nx_off1 = 0;
    if (H1 && c < c_end) {
        nx_end1 = load_sub_end(sec1 + tab_sub, sub_w, c, lane);
        nx_off1 = reinterpret_cast<const uint32_t*>(sec1 + tab_chunk)[c];
    }

    // The pieces of one chunk at a time live in the warp's staging slots.  A chunk's pieces are requested as soon
    // as the chunk before it has been decoded (the slots are free then), so the copy runs while that chunk is
    // merged and written.  State of the chunk whose pieces are in the slots or on their way:
    uint32_t end0 = 0, end1 = 0, start0 = 0, start1 = 0, piece0 = 0, piece1 = 0;
    const uint32_t* pay0_g = nullptr;
    const uint32_t* pay1_g = nullptr;
    bool staged0 = false, staged1 = false, flying0 = false, flying1 = false;
    // Sliced pieces: bits of the piece before the current slice (rel), position at the slice's start (org), and the
    // slice that is on its way: its bytes per lane (by), where it starts in the piece (at), bytes of the whole warp (tot).
    uint32_t rel0 = 0, rel1 = 0, org0 = 0, org1 = 0;
    uint32_t by0 = 0, by1 = 0, at0 = 0, at1 = 0, tot0 = 0, tot1 = 0;
    // Every lane fetches the next slice of its own subchunk, from bit rel of the piece on: 16-byte aligned, long
    // enough for kSliceSyms symbols of 12 bits plus the window's look-ahead, not past the piece's guard (with a
    // damaged payload a lane may have run past its piece: the copy still stays inside piece + guard).  The copies
    // are waited for when the slice is needed; until then the warp merges and writes the symbols it has.
    auto issue_slices = [&](const bool more0, const bool more1) {
        by0 = by1 = 0;
        at0 = min(16 * (rel0 >> 7), piece0); at1 = min(16 * (rel1 >> 7), piece1);
        if (H0 && sliced0 && more0) by0 = min(kSliceBytes, piece0 + 16 - at0);
        if (H1 && sliced1 && more1) by1 = min(kSliceBytes, piece1 + 16 - at1);
        tot0 = H0 ? __reduce_add_sync(0xFFFFFFFFu, by0) : 0u;
        tot1 = H1 ? __reduce_add_sync(0xFFFFFFFFu, by1) : 0u;
        __syncwarp();                                            // every lane is done with the previous slices
        if (tot0) flying0 = true;
        if (tot1) flying1 = true;
        if (P.skip_copy) return;
        if (lane == 0) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            if (tot0) mbar_expect_tx(&bar[0], tot0);
            if (tot1) mbar_expect_tx(&bar[1], tot1);
        }
        __syncwarp();
        if (by0) bulk_g2s_addr(slot0_s, reinterpret_cast<const uint8_t*>(pay0_g) + at0, by0, &bar[0]);
        if (by1) bulk_g2s_addr(slot1_s, reinterpret_cast<const uint8_t*>(pay1_g) + at1, by1, &bar[1]);
    };
    // Takes the table entries in nx_* (of chunk `cc`), checks them, starts the copies, and requests the entries
    // of the chunk after it.
    auto prepare = [&](const uint32_t cc) {
        bool ok = true;
        if (H0) {
            const uint32_t off16 = nx_off0;
            end0 = nx_end0;
            start0 = __shfl_up_sync(0xFFFFFFFFu, end0, 1);
            if (lane == 0) start0 = 0;
            const uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, end0, 31);
            piece0 = ((chunk_bits + 127) / 128) * 16;
            ok = ok && start0 <= end0 && end0 - start0 <= P.sub * kLmax && (uint64_t)off16 + piece0 / 16 <= payload16;
            pay0_g = reinterpret_cast<const uint32_t*>(payload + 16ull * off16);
        }
        if (H1) {
            const uint32_t off16 = nx_off1;
            end1 = nx_end1;
            start1 = __shfl_up_sync(0xFFFFFFFFu, end1, 1);
            if (lane == 0) start1 = 0;
            const uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, end1, 31);
            piece1 = ((chunk_bits + 127) / 128) * 16;
            ok = ok && start1 <= end1 && end1 - start1 <= P.sub * kLmax && (uint64_t)off16 + piece1 / 16 <= payload16;
            pay1_g = reinterpret_cast<const uint32_t*>(payload + 16ull * off16);
        }
        staged0 = staged1 = false;
        if (kHuff && !__all_sync(0xFFFFFFFFu, ok)) { err = ZC_E_CORRUPT; return; }
        // the copy takes 16 bytes more than the piece (the next piece or the guard), so window peeks stay inside
        sliced0 = H0 && can_slice && piece0 + 16 > slot_bytes;
        sliced1 = H1 && can_slice && piece1 + 16 > slot_bytes;
        slot0_s = base0_s + (sliced0 ? lane * kSliceSlot : 0u);
        slot1_s = base1_s + (sliced1 ? lane * kSliceSlot : 0u);
        if (sliced0) staged0 = true;
        if (sliced1) staged1 = true;
        if (sliced0 || sliced1) {
            rel0 = start0; rel1 = start1;
            issue_slices(end0 > start0, end1 > start1);          // lanes that have bits at all
        }
        if (H0 && piece0 + 16 <= slot_bytes) {
            staged0 = flying0 = true;
            if (lane == 0 && !P.skip_copy) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_expect_tx(&bar[0], piece0 + 16);
                bulk_g2s(pool + slots_off, pay0_g, piece0 + 16, &bar[0]);
            }
        }
        if (H1 && piece1 + 16 <= slot_bytes) {
            staged1 = flying1 = true;
            if (lane == 0 && !P.skip_copy) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_expect_tx(&bar[1], piece1 + 16);
                bulk_g2s(pool + slots_off + (H0 ? slot_bytes : 0), pay1_g, piece1 + 16, &bar[1]);
            }
        }
        const uint32_t cn = cc + step;
        if (cn < c_end) {
            if (H0) { nx_end0 = load_sub_end(sec0 + tab_sub, sub_w, cn, lane);
                      nx_off0 = reinterpret_cast<const uint32_t*>(sec0 + tab_chunk)[cn]; }
            if (H1) { nx_end1 = load_sub_end(sec1 + tab_sub, sub_w, cn, lane);
                      nx_off1 = reinterpret_cast<const uint32_t*>(sec1 + tab_chunk)[cn]; }
        }
    };
    if (c < c_end) prepare(c);

    for (; c < c_end && !err; c += step) {
        // ---- the chunk; FULL: a complete chunk, every lane has P.sub symbols ----
        auto body = [&](auto full_tag) {
            constexpr bool FULL = decltype(full_tag)::value;
            const uint64_t c_lo = (uint64_t)c * P.cs;
            const uint32_t c_syms = FULL ? P.cs : (uint32_t)min((uint64_t)P.cs, P.n_syms - c_lo);
            const uint32_t out_bytes = FULL ? P.chunk_bytes : (uint32_t)min((uint64_t)P.chunk_bytes, P.input_bytes - 2 * c_lo);
            const uint32_t lo_sym = lane * P.sub;
            const uint32_t n_my = FULL ? P.sub : (lo_sym < c_syms ? min(P.sub, c_syms - lo_sym) : 0u);
            const uint32_t last_r = FULL ? n_rounds - 1 : (min(c_syms, P.sub) - 1) / R;   // lane 0 has the most symbols
            const uint8_t* raw0 = sec0 + c_lo + k_lane;             // my first part's bytes in a raw stream
            const uint8_t* raw1 = sec1 + c_lo + k_lane;
            uint8_t* dst_lane = P.out + 2 * c_lo + 2 * k_lane;      // two element bytes per symbol in every format
            uint32_t pos0 = 0, pos1 = 0, w00 = 0, w01 = 0, w10 = 0, w11 = 0, next0 = 0, next1 = 0;
            uint32_t lim0 = 0, lim1 = 0;
            for (uint32_t r = 0; r <= last_r; ++r) {
                // ---- raw sign+mantissa bytes of this round go to registers before the decoding starts ----
#pragma unroll
                for (int i = 0; i < PPL; ++i)
                    if (!H1 && (FULL || k_lane + i * k_step + r * R < c_syms))
                        asm volatile("prefetch.global.L2 [%0];" :: "l"(raw1 + i * k_step + r * R));
                if (kHuff && (sliced0 || sliced1) && r % kRoundsPerSlice == 0) {
                    // the slice requested after the previous one was used up (or, for the chunk's first one, while
                    // the chunk before was merged) is needed now
                    if (tot0) { if (mbar_wait(&bar[0], parity0, P.spin_limit)) { parity0 ^= 1; flying0 = false; } else err = ZC_E_DEVICE_TIMEOUT; }
                    if (tot1) { if (mbar_wait(&bar[1], parity1, P.spin_limit)) { parity1 ^= 1; flying1 = false; } else err = ZC_E_DEVICE_TIMEOUT; }
                    if (__any_sync(0xFFFFFFFFu, err == ZC_E_DEVICE_TIMEOUT)) { err = ZC_E_DEVICE_TIMEOUT; return; }
                    if (by0) { org0 = 8 * slot0_s + min(rel0 - 8 * at0, 127u); lane_start(pos0, w00, w01, next0, org0); }
                    if (by1) { org1 = 8 * slot1_s + min(rel1 - 8 * at1, 127u); lane_start(pos1, w10, w11, next1, org1); }
                    tot0 = tot1 = 0;
                }
                if (kHuff && r == 0) {
                    if (H0 && staged0 && !sliced0) {
                        if (mbar_wait(&bar[0], parity0, P.spin_limit)) parity0 ^= 1; else err = ZC_E_DEVICE_TIMEOUT;
                    }
                    if (H1 && staged1 && !sliced1) {
                        if (mbar_wait(&bar[1], parity1, P.spin_limit)) parity1 ^= 1; else err = ZC_E_DEVICE_TIMEOUT;
                    }
                    if (__any_sync(0xFFFFFFFFu, err == ZC_E_DEVICE_TIMEOUT)) { err = ZC_E_DEVICE_TIMEOUT; return; }
                    if (!sliced0) flying0 = false;
                    if (!sliced1) flying1 = false;
                    // staged: positions count from shared address 0; from global memory: from the piece, and the last
                    // readable word pair ends with the guard (piece + 16 bytes)
                    if (H0 && !sliced0) { if (staged0) lane_start(pos0, w00, w01, next0, 8 * slot0_s + start0); else pos0 = start0; lim0 = piece0 / 4 + 2; }
                    if (H1 && !sliced1) { if (staged1) lane_start(pos1, w10, w11, next1, 8 * slot1_s + start1); else pos1 = start1; lim1 = piece1 / 4 + 2; }
                }
                // ---- every lane decodes R symbols of its subchunk ----
                if (kHuff) {
                    const uint32_t done = r * R;
                    // a ragged end decodes up to 15 symbols too many (from the bits that follow); they are not used
                    const uint32_t n_quads = FULL ? (uint32_t)PPL : (n_my > done ? (min(R, n_my - done) + 15) / 16 : 0u);
                    // (only in the kernels built for launches that expect two coded streams: they have the registers for it)
                    constexpr bool kSideBySide = H0 && H1 && (XOR || FMT == ZC_FMT_SCALE_U8);
                    if (kSideBySide && n_quads && staged0 && staged1 && piece0 != 0 && piece1 != 0) {
                        // both streams come from staged pieces: their words are decoded side by side
                        const uint32_t wra_s = rows0_s + wr_off, wrb_s = rows1_s + wr_off;
                        if (S.pairs0) {
                            if (S.pairs1) decode_round2<2, 2, PPL, FULL>(pos0, w00, w01, next0, S.lut0_s, wra_s, pos1, w10, w11, next1, S.lut1_s, wrb_s, fw, n_quads);
                            else decode_round2<2, 1, PPL, FULL>(pos0, w00, w01, next0, S.lut0_s, wra_s, pos1, w10, w11, next1, S.lut1_s, wrb_s, fw, n_quads);
                        } else {
                            if (S.pairs1) decode_round2<1, 2, PPL, FULL>(pos0, w00, w01, next0, S.lut0_s, wra_s, pos1, w10, w11, next1, S.lut1_s, wrb_s, fw, n_quads);
                            else decode_round2<1, 1, PPL, FULL>(pos0, w00, w01, next0, S.lut0_s, wra_s, pos1, w10, w11, next1, S.lut1_s, wrb_s, fw, n_quads);
                        }
                    } else if (n_quads) {
                        if (H0) {
                            const uint32_t wr_s = rows0_s + wr_off;
                            if (piece0 == 0) fill_quads(S.lut0_s, S.pairs0, wr_s, fw, n_quads);   // a chunk without bits: nothing but the fill symbol
                            else if (!staged0) pos0 = decode_quads_global(pos0, pay0_g, S.lut0_s, S.pairs0, wr_s, fw, n_quads, lim0);
                            else if (S.pairs0) decode_round<2, PPL, FULL>(pos0, w00, w01, next0, S.lut0_s, wr_s, fw, n_quads);
                            else decode_round<1, PPL, FULL>(pos0, w00, w01, next0, S.lut0_s, wr_s, fw, n_quads);
                        }
                        if (H1) {
                            const uint32_t wr_s = rows1_s + wr_off;
                            if (piece1 == 0) fill_quads(S.lut1_s, S.pairs1, wr_s, fw, n_quads);
                            else if (!staged1) pos1 = decode_quads_global(pos1, pay1_g, S.lut1_s, S.pairs1, wr_s, fw, n_quads, lim1);
                            else if (S.pairs1) decode_round<2, PPL, FULL>(pos1, w10, w11, next1, S.lut1_s, wr_s, fw, n_quads);
                            else decode_round<1, PPL, FULL>(pos1, w10, w11, next1, S.lut1_s, wr_s, fw, n_quads);
                        }
                    }
                    __syncwarp();
                    if ((sliced0 || sliced1) && (r + 1) % kRoundsPerSlice == 0 && r < last_r) {
                        if (sliced0) { rel0 += pos0 - org0; org0 = pos0; }
                        if (sliced1) { rel1 += pos1 - org1; org1 = pos1; }
                        issue_slices(n_my > (r + 1) * R, n_my > (r + 1) * R);
                    }
                    if (r == last_r) {
                        // Every lane must have consumed exactly the bits of its subchunk (a ragged end decodes up to
                        // fifteen symbols too many).  Anything else means the payload does not belong to the tables.
                        bool good = true;
                        if (H0) {
                            const uint32_t used = sliced0 ? rel0 + pos0 - org0 : pos0 - (staged0 ? 8 * slot0_s : 0u);
                            good = good && (FULL ? used == end0 : used - end0 <= 15 * kLmax);
                        }
                        if (H1) {
                            const uint32_t used = sliced1 ? rel1 + pos1 - org1 : pos1 - (staged1 ? 8 * slot1_s : 0u);
                            good = good && (FULL ? used == end1 : used - end1 <= 15 * kLmax);
                        }
                        if (!__all_sync(0xFFFFFFFFu, good)) err = ZC_E_CORRUPT;
                        // the slots are free: the next chunk's pieces travel while this round is merged and written
                        if (!err && c + step < c_end) prepare(c + step);
                    }
                }
                // ---- cooperative merge: a part covers 16 symbols = 32 output bytes ----
#pragma unroll
                for (int i = 0; i < PPL; ++i) {
                    const uint32_t k = k_lane + i * k_step + r * R;
                    if ((!FULL && k >= c_syms)) continue;
                    uint32_t e[4], m[4];
                    if (H0) {
                        const uint4 v = lds128(rows0_s + rd_off + 512 * i);
                        e[0] = v.x; e[1] = v.y; e[2] = v.z; e[3] = v.w;
                    } else {
                        const uint4 v = ld_nc_v4(raw0 + i * k_step + r * R);
                        e[0] = v.x; e[1] = v.y; e[2] = v.z; e[3] = v.w;
                    }
                    if (H1) {
                        const uint4 v = lds128(rows1_s + rd_off + 512 * i);
                        m[0] = v.x; m[1] = v.y; m[2] = v.z; m[3] = v.w;
                    } else {
                        const uint4 v = ld_nc_v4(raw1 + i * k_step + r * R);
                        m[0] = v.x; m[1] = v.y; m[2] = v.z; m[3] = v.w;
                    }
                    uint32_t o[8];
                    merge16<FMT>(e, m, o);
                    merge16<FMT>(e + 2, m + 2, o + 4);
                    uint8_t* dst = dst_lane + 2 * (i * k_step + r * R);
                    if (XOR && P.base) {                              // delta form: XOR the base tensor back in
                        const uint64_t off = (uint64_t)(dst - P.out);
                        const uint4 b0 = load16_guarded(P.base, off, P.input_bytes), b1 = load16_guarded(P.base, off + 16, P.input_bytes);
                        o[0] ^= b0.x; o[1] ^= b0.y; o[2] ^= b0.z; o[3] ^= b0.w;
                        o[4] ^= b1.x; o[5] ^= b1.y; o[6] ^= b1.z; o[7] ^= b1.w;
                    }
                    if (FULL || 2 * k + 32 <= out_bytes) {
                        st_cs_v8(dst, o);
                    } else {
#pragma unroll
                        for (int t = 0; t < 32; ++t)
                            if (2 * k + t < out_bytes) dst[t] = (uint8_t)(o[t >> 2] >> (8 * (t & 3)));
                    }
                }
                if (kHuff) __syncwarp();
            }
        };
        if (c < n_full) body(BoolTag<true>{}); else body(BoolTag<false>{});
    }
    // a copy that was started and not waited for (the loop ended early) must land before the block may leave
    if (flying0 && !P.skip_copy) mbar_wait(&bar[0], parity0, P.spin_limit);
    if (flying1 && !P.skip_copy) mbar_wait(&bar[1], parity1, P.spin_limit);
    return err;
}

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
// PPL = 16-symbol parts each lane merges per round = R / 16, R in {16, 32, 64}.

struct DecSmem {                     // the block's dynamic shared memory, carved up once per kernel
    uint32_t* lut0;                  // decode table of stream 0
    uint32_t* lut1;                  // decode table of stream 1
    uint32_t* scratch;
    uint8_t* pools;                  // all warps' pools
    uint8_t* pool;                   // this warp's pool
    uint64_t* bar;                   // this warp's two mbarriers
};

__device__ __forceinline__ DecSmem carve_smem(uint8_t* smem, uint32_t pool_bytes)
{
    const uint32_t warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    DecSmem m;
    m.lut0 = reinterpret_cast<uint32_t*>(smem);
    m.lut1 = reinterpret_cast<uint32_t*>(smem + kLutBytes);
    m.scratch = reinterpret_cast<uint32_t*>(smem + 2 * kLutBytes);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kDecFixedSmem);
    m.pools = reinterpret_cast<uint8_t*>(bars + 2 * n_warps);
    m.pool = m.pools + (size_t)warp * pool_bytes;
    m.bar = bars + 2 * warp;
    if ((threadIdx.x & 31) == 0) { mbar_init(&m.bar[0], 1); mbar_init(&m.bar[1], 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    return m;
}

// Decodes the chunks c0, c0 + step, ... (< c_end) of one tensor with this warp; the whole block calls it
// together (the header check and the table build are block-wide).  Returns a zc_status, the same in every
// thread for the block-wide checks.
template <int FMT, int PPL, bool XOR>
__device__ __forceinline__ uint32_t decode_one(const DecParams& P, const DecSmem& M, const uint32_t chunk_base, const uint32_t c_end,
                                               const uint32_t block_index, const uint32_t n_blocks, uint32_t& parity0, uint32_t& parity1)
{
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    // chunk chunk_base + k goes to block (k / n_warps) % n_blocks, warp k % n_warps
    uint32_t c0 = chunk_base + block_index * n_warps + warp, step = n_blocks * n_warps;
    const uint32_t sub_w = P.chunk_bytes <= 8192 ? 2u : 4u;     // bytes per sub_end entry
    const uint64_t tab_chunk = 256, tab_sub = 256 + (((uint64_t)4 * P.n_chunks + 15) & ~15ull);
    // Nearly every container has stream 0 coded, its table section right behind the header.  Its code lengths
    // and this warp's first table entries are requested now, together with the header, and thrown away if the
    // header says otherwise.
    uint32_t spec_len = 0, spec_end = 0, spec_off = 0;
    if (P.spec) {
        if (threadIdx.x < 256) spec_len = P.comp[kHeaderBytes + threadIdx.x];
        if (c0 < c_end) {
            spec_end = load_sub_end(P.comp + kHeaderBytes + tab_sub, sub_w, c0, lane);
            spec_off = reinterpret_cast<const uint32_t*>(P.comp + kHeaderBytes + tab_chunk)[c0];
        }
    }
    // ---- header check against the plan ----
    __shared__ uint32_t s_mode[2], s_per_lookup[2];
    __shared__ uint32_t s_ok;
    __shared__ unsigned long long s_payload_off, s_payload_bytes, s_sec[2];
    __shared__ __align__(16) uint32_t s_hdr[32];
    if (warp == 0) {
        s_hdr[lane] = reinterpret_cast<const uint32_t*>(P.comp)[lane];      // the 128-byte header in one request
        __syncwarp();
    }
    if (threadIdx.x == 0) {
        const uint8_t* h = reinterpret_cast<const uint8_t*>(s_hdr);
        const uint32_t* h32 = s_hdr;
        const unsigned long long* h64 = reinterpret_cast<const unsigned long long*>(s_hdr);
        bool ok = h32[0] == kMagic && h[kHdrVersion] == 1 && h[kHdrVersion + 1] == 0 && h[kHdrFormat] == P.format &&
                  h[kHdrStreams] == 2 && h64[kHdrElems / 8] == P.n_elems && h32[kHdrChunkBytes / 4] == P.chunk_bytes &&
                  h32[kHdrChunks / 4] == P.n_chunks && h[kHdrLmax] == kLmax && h[kHdrGroup] == P.group && h[kHdrSubs] == kSubs &&
                  h[kHdrSubWidth] == sub_w;
        uint32_t mode[2] = {0, 0};
        for (int s = 0; s < 2 && ok; ++s) {
            const uint8_t* d = h + kHdrStream0 + kHdrStreamStride * s;
            mode[s] = d[kSdMode];
            ok = mode[s] <= 1 && reinterpret_cast<const unsigned long long*>(d)[1] == P.n_syms;
        }
        if (ok) {
            // recompute where everything must be and compare with what the header says
            uint64_t off = kHeaderBytes, sec[2] = {0, 0};
            const uint64_t tab = 256 + (((uint64_t)4 * P.n_chunks + 15) & ~15ull) + 32ull * sub_w * P.n_chunks;
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
    __syncthreads();
    if (!s_ok) return ZC_E_CORRUPT;

    const bool huff0 = s_mode[0] == ZC_MODE_HUFF, huff1 = s_mode[1] == ZC_MODE_HUFF;
    {
        // the warps' pools are free until the chunk loop: 8 KiB of them hold the one-symbol scratch table
        uint16_t* single = reinterpret_cast<uint16_t*>(M.pools);
        bool tables_ok = true;
        if (huff0) {
            uint32_t len = spec_len;                             // stream 0's section always starts behind the header
            if (!P.spec && threadIdx.x < 256) len = P.comp[s_sec[0] + threadIdx.x];
            tables_ok = build_lut(len, M.lut0, single, M.scratch, &s_per_lookup[0]) && tables_ok;
        }
        if (huff1) {
            uint32_t len = 0;
            if (threadIdx.x < 256) len = P.comp[s_sec[1] + threadIdx.x];
            tables_ok = build_lut(len, M.lut1, single, M.scratch, &s_per_lookup[1]) && tables_ok;
        }
        __syncthreads();
        if (!tables_ok) return ZC_E_CORRUPT;
    }

    // Large chunks with both streams coded: a warp's pool was sized for one coded stream's lane slots (the plan
    // does not say how many streams a container codes); fewer warps then share the block's pools, each with room
    // for both, and the chunks are dealt to those warps only.
    uint8_t* pool = M.pool;
    uint32_t pool_bytes = P.pool_bytes;
    if (P.sliced && huff0 && huff1) {
        const uint32_t need = 2 * (512 * PPL + 32 * kSliceSlot);
        if (need > P.pool_bytes) {
            const uint32_t active = max(1u, n_warps * P.pool_bytes / need);
            pool = M.pools + (size_t)min(warp, active - 1) * need;
            pool_bytes = need;
            c0 = warp < active ? chunk_base + block_index * active + warp : c_end;
            step = n_blocks * active;
            spec_end = spec_off = 0;
            if (c0 < c_end) {
                spec_end = load_sub_end(P.comp + kHeaderBytes + tab_sub, sub_w, c0, lane);
                spec_off = reinterpret_cast<const uint32_t*>(P.comp + kHeaderBytes + tab_chunk)[c0];
            }
        }
    }
    DecShared S;
    S.pool_bytes = pool_bytes;
    S.lut0_s = smem_u32(M.lut0); S.lut1_s = smem_u32(M.lut1);
    S.pairs0 = huff0 && s_per_lookup[0] == 2;
    S.pairs1 = huff1 && s_per_lookup[1] == 2;
    S.sec0 = s_sec[0]; S.sec1 = s_sec[1];
    S.payload_off = s_payload_off; S.payload_bytes = s_payload_bytes;
    uint32_t first_end0 = spec_end, first_off0 = spec_off;
    if (huff0 && !P.spec && c0 < c_end) {
        first_end0 = load_sub_end(P.comp + S.sec0 + tab_sub, sub_w, c0, lane);
        first_off0 = reinterpret_cast<const uint32_t*>(P.comp + S.sec0 + tab_chunk)[c0];
    }
    if (huff0 && !huff1) return run_chunks<FMT, PPL, true, false, XOR>(P, S, pool, M.bar, first_end0, first_off0, c0, c_end, step, parity0, parity1);
    if (!huff0 && !huff1) return run_chunks<FMT, PPL, false, false, XOR>(P, S, pool, M.bar, 0, 0, c0, c_end, step, parity0, parity1);
    if (huff0) return run_chunks<FMT, PPL, true, true, XOR>(P, S, pool, M.bar, first_end0, first_off0, c0, c_end, step, parity0, parity1);
    return run_chunks<FMT, PPL, false, true, XOR>(P, S, pool, M.bar, 0, 0, c0, c_end, step, parity0, parity1);
}

// One tensor per launch: the warps of all blocks take the chunks in turn.
template <int FMT, int PPL>
__global__ void __launch_bounds__(dec_block_warps<FMT, false>() * 32, 1)
decode_kernel(const __grid_constant__ DecParams P)
{
    extern __shared__ __align__(16) uint8_t smem[];
    const DecSmem M = carve_smem(smem, P.pool_bytes);
    if (P.ctl && blockIdx.x == 0 && threadIdx.x == 0) P.ctl->call_id = P.call_id;
    uint32_t parity0 = 0, parity1 = 0;
    const uint32_t err = decode_one<FMT, PPL, false>(P, M, P.c_begin, P.c_end, blockIdx.x, gridDim.x, parity0, parity1);
    if (err) raise_status(P.ctl, P.call_id, err);
}

// Many tensors per launch: block b takes the chunks [b * total / grid, (b + 1) * total / grid) of the
// concatenated chunk index space, tensor by tensor; it builds the tables of a tensor once for its whole share.
// XOR: the launch has base tensors (delta form); a kernel of its own so that the plain form pays nothing for it.
template <int FMT, int PPL, bool XOR>
__global__ void __launch_bounds__(dec_block_warps<FMT, XOR>() * 32, 1)
decode_batch_kernel(const __grid_constant__ DecBatchParams B)
{
    extern __shared__ __align__(16) uint8_t smem[];
    const DecSmem M = carve_smem(smem, B.pool_bytes);
    if (blockIdx.x == 0 && threadIdx.x == 0 && B.tensor_base == 0) B.ctl->call_id = B.call_id;
    uint32_t parity0 = 0, parity1 = 0;

    auto run = [&](const uint32_t t, const uint32_t seg_lo, const uint32_t seg_hi) {
        DecParams P;
        P.comp = B.item[t].comp; P.base = XOR ? B.item[t].base : nullptr; P.out = B.item[t].out; P.ctl = B.ctl;
        P.comp_bytes = B.item[t].comp_bytes; P.input_bytes = B.item[t].input_bytes;
        P.n_syms = B.item[t].n_syms; P.n_elems = B.item[t].n_elems; P.n_chunks = B.item[t].n_chunks;
        P.cs = B.cs; P.sub = B.sub; P.chunk_bytes = B.chunk_bytes; P.format = B.format; P.group = B.group;
        P.pool_bytes = B.pool_bytes; P.call_id = B.call_id; P.c_begin = 0; P.c_end = P.n_chunks;
        P.spin_limit = B.spin_limit; P.skip_copy = B.skip_copy; P.sliced = B.sliced;
        const uint64_t tables = 256 + (((uint64_t)4 * P.n_chunks + 15) & ~15ull) + 32ull * (P.chunk_bytes <= 8192 ? 2u : 4u) * P.n_chunks;
        P.spec = P.comp_bytes >= kHeaderBytes + tables ? 1u : 0u;
        __syncthreads();                                         // everybody is done with the previous tensor's tables
        const uint32_t err = decode_one<FMT, PPL, XOR>(P, M, seg_lo, seg_hi, 0, 1, parity0, parity1);
        if (err && raise_status(B.ctl, B.call_id, err)) B.ctl->failed = B.tensor_base + t + 1;
    };

    // The concatenated chunk index space is cut into n_ranges equal ranges which the blocks take one after the
    // other from a ticket counter (tensors, and SMs, differ in how fast they get through a range).  Block 0
    // first walks over the tensors without chunks: their headers are still checked.
    __shared__ uint32_t s_range;
    uint32_t empties = blockIdx.x == 0 ? 0u : B.n_tensors;      // cursor of that walk
    uint32_t t = 0, g = 0, g_hi = 0;
    bool in_range = false;
    for (;;) {
        uint32_t tt, seg_lo, seg_hi;
        if (empties < B.n_tensors) {
            if (B.item[empties].n_chunks != 0) { ++empties; continue; }
            tt = empties++; seg_lo = 0; seg_hi = 0;
        } else {
            if (!in_range) {
                __syncthreads();
                if (threadIdx.x == 0) s_range = atomicAdd(&B.ctl->ticket, 1u);
                __syncthreads();
                const uint32_t r = s_range;
                if (r >= B.n_ranges) break;
                g = (uint32_t)((uint64_t)r * B.total_chunks / B.n_ranges);
                g_hi = (uint32_t)((uint64_t)(r + 1) * B.total_chunks / B.n_ranges);
                // the last tensor that starts at or before g (tensors without chunks share their start with the next one)
                uint32_t lo = 0, hi = B.n_tensors;
                while (hi - lo > 1) {
                    const uint32_t mid = (lo + hi) / 2;
                    if (B.item[mid].first_chunk <= g) lo = mid; else hi = mid;
                }
                t = lo;
                in_range = true;
            }
            if (g >= g_hi || t >= B.n_tensors) { in_range = false; continue; }
            const uint32_t first = B.item[t].first_chunk, n = B.item[t].n_chunks;
            if (g >= first + n) { ++t; continue; }
            seg_hi = min(g_hi, first + n) - first;
            seg_lo = g - first;
            tt = t++;
            g = first + seg_hi;
        }
        run(tt, seg_lo, seg_hi);
    }
}


// ---- launchers, one set per element format -------------------------------------------------------------------
// The kernels of one format are instantiated where that format's launchers are defined.  This file can be compiled
// as a whole (ZC_DEC_PART undefined or 0) or in four parts (1: the C ABI and BF16, 2: FP8, 3: scale bytes, 4: FP4), one
// object each, so that a build compiles the formats side by side.
#ifndef ZC_DEC_PART
#define ZC_DEC_PART 0
#endif

// the buffers of a launch, for the development build's checks
struct DecRanges { const void* in; size_t in_bytes; const void* out; size_t out_bytes; const void* ws; size_t ws_bytes; };

template <int F>
cudaError_t dec_launch_single_t(uint32_t ppl, uint32_t grid, uint32_t threads, size_t smem, cudaStream_t st, const DecParams& P,
                                const DecRanges& R)
{
    cudaError_t e = cudaSuccess;
    auto launch = [&](auto kern) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return;
#if ZC_DEBUG_CHECKS
        dbg_set_ranges(st, R.in, R.in_bytes, R.out, R.out_bytes, R.ws, R.ws_bytes);
#else
        (void)R;
#endif
        kern<<<grid, threads, smem, st>>>(P);
        e = cudaGetLastError();
    };
    if (ppl == 4) launch(decode_kernel<F, 4>);
    else if (ppl == 2) launch(decode_kernel<F, 2>);
    else launch(decode_kernel<F, 1>);
    return e;
}

template <int F>
cudaError_t dec_launch_batch_t(uint32_t ppl, bool any_base, uint32_t grid, uint32_t threads, size_t smem, cudaStream_t st,
                               const DecBatchParams& B, const DecRanges& R)
{
    cudaError_t e = cudaSuccess;
    auto launch = [&](auto kern) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return;
#if ZC_DEBUG_CHECKS
        dbg_set_ranges(st, R.in, R.in_bytes, R.out, R.out_bytes, R.ws, R.ws_bytes);
#else
        (void)R;
#endif
        kern<<<grid, threads, smem, st>>>(B);
        e = cudaGetLastError();
    };
    if (any_base) {
        if (ppl == 4) launch(decode_batch_kernel<F, 4, true>);
        else if (ppl == 2) launch(decode_batch_kernel<F, 2, true>);
        else launch(decode_batch_kernel<F, 1, true>);
    } else {
        if (ppl == 4) launch(decode_batch_kernel<F, 4, false>);
        else if (ppl == 2) launch(decode_batch_kernel<F, 2, false>);
        else launch(decode_batch_kernel<F, 1, false>);
    }
    return e;
}

#define ZC_DEC_DECLARE(NAME)                                                                                              \
    cudaError_t dec_launch_single_##NAME(uint32_t ppl, uint32_t grid, uint32_t threads, size_t smem, cudaStream_t st,     \
                                         const DecParams& P, const DecRanges& R);                                        \
    cudaError_t dec_launch_batch_##NAME(uint32_t ppl, bool any_base, uint32_t grid, uint32_t threads, size_t smem,        \
                                        cudaStream_t st, const DecBatchParams& B, const DecRanges& R);                   \
    void dec_debug_counts_##NAME(uint32_t out[2]);
ZC_DEC_DECLARE(bf16)
ZC_DEC_DECLARE(fp8)
ZC_DEC_DECLARE(scale)
ZC_DEC_DECLARE(fp4)
#undef ZC_DEC_DECLARE

#if ZC_DEBUG_CHECKS
#define ZC_DEC_COUNTS(out) dbg_read_counts(out)
#else
#define ZC_DEC_COUNTS(out) (void)(out)
#endif
#define ZC_DEC_DEFINE(NAME, F)                                                                                            \
    cudaError_t dec_launch_single_##NAME(uint32_t ppl, uint32_t grid, uint32_t threads, size_t smem, cudaStream_t st,     \
                                         const DecParams& P, const DecRanges& R)                                         \
    { return dec_launch_single_t<F>(ppl, grid, threads, smem, st, P, R); }                                                \
    cudaError_t dec_launch_batch_##NAME(uint32_t ppl, bool any_base, uint32_t grid, uint32_t threads, size_t smem,        \
                                        cudaStream_t st, const DecBatchParams& B, const DecRanges& R)                    \
    { return dec_launch_batch_t<F>(ppl, any_base, grid, threads, smem, st, B, R); }                                       \
    void dec_debug_counts_##NAME(uint32_t out[2]) { ZC_DEC_COUNTS(out); }
#if ZC_DEC_PART == 0 || ZC_DEC_PART == 1
ZC_DEC_DEFINE(bf16, ZC_FMT_BF16)
#endif
#if ZC_DEC_PART == 0 || ZC_DEC_PART == 2
ZC_DEC_DEFINE(fp8, ZC_FMT_FP8_E4M3)
#endif
#if ZC_DEC_PART == 0 || ZC_DEC_PART == 3
ZC_DEC_DEFINE(scale, ZC_FMT_SCALE_U8)
#endif
#if ZC_DEC_PART == 0 || ZC_DEC_PART == 4
ZC_DEC_DEFINE(fp4, ZC_FMT_FP4_E2M1)
#endif
#undef ZC_DEC_DEFINE

}  // namespace zc

#if ZC_DEC_PART <= 1

using namespace zc;

extern "C" {

namespace {

// Launch shape for a plan: symbols per round and lane, per-warp pool, warps per block, shared memory.
struct DecShape { uint32_t ppl, pool_bytes, warps, sliced; size_t smem; };

// both_coded: expect both streams to be Huffman-coded (scale bytes, deltas) instead of one
zc_status dec_shape(const zc_plan_t* p, bool both_coded, DecShape* out)
{
    DecShape s{};
    // symbols per round and lane: the largest of 64 / 32 / 16 that divides the subchunk length
    s.ppl = (p->syms_per_sub % 64 == 0) ? 4 : (p->syms_per_sub % 32 == 0) ? 2 : 1;
    // scale bytes and deltas have both streams coded as a rule, plain tensors one (the other one is raw)
    const uint32_t coded = (both_coded || p->format == ZC_FMT_SCALE_U8) ? 2 : 1;
    const uint32_t rows_bytes = 512 * s.ppl;
    // per warp: the coded streams' rows plus room to stage, per coded stream, a piece as large as the raw chunk
    // stream; pieces that do not fit (or chunks above 16 KiB of symbols) are read from global memory instead
    s.sliced = p->syms_per_sub % kSliceSyms == 0 ? 1u : 0u;   // pieces beyond their slot can be staged slice by slice
    s.pool_bytes = std::max<uint32_t>(coded * (rows_bytes + std::min<uint32_t>(p->syms_per_chunk, 16384) + 32), 2 * rows_bytes);
    // chunks above 16 KiB: whole pieces would leave room for a dozen warps at most; lane slots for sliced pieces
    // are enough, and more warps decode
    if (s.sliced && p->syms_per_chunk > 8192) s.pool_bytes = std::max<uint32_t>(coded * (rows_bytes + 32 * kSliceSlot), 2 * rows_bytes);
    // slack behind the last slot: what a lane can read past its piece when the payload is damaged (see window_s)
    const size_t slack = (size_t)round_up(p->syms_per_sub + p->syms_per_sub / 2 + 16, 16);
    const size_t fixed = kDecFixedSmem + 512 /* static shared */ + slack;
    size_t per_warp = 16 + s.pool_bytes;
    const size_t max_warps = coded == 2 ? kDecMaxWarpsBoth : kDecMaxWarps;     // the kernels' launch bounds
    s.warps = (uint32_t)std::min<size_t>(max_warps, (kMaxSmem - fixed - 1024) / per_warp);
    if (s.warps < 8) {               // large chunks: stage less
        s.pool_bytes = std::max<uint32_t>(coded * (rows_bytes + 32 * kSliceSlot), 2 * rows_bytes);   // room for the lane slots of sliced pieces
        per_warp = 16 + s.pool_bytes;
        s.warps = (uint32_t)std::min<size_t>(max_warps, (kMaxSmem - fixed - 1024) / per_warp);
    }
    // the table build uses 8 KiB of the pools and 256 threads
    while (s.warps * (size_t)s.pool_bytes < 8192) ++s.warps;
    if (s.warps < 8 || s.warps > max_warps) return ZC_E_UNSUPPORTED;
    s.smem = kDecFixedSmem + s.warps * per_warp + slack;
    *out = s;
    return ZC_OK;
}

// no clearing of the workspace: errors are tagged with the id of the call that raised them
unsigned long long new_call_id()
{
    static std::atomic<unsigned long long> next_call{(unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count()};
    return (next_call.fetch_add(1) & ((1ull << 56) - 1)) | 1ull << 55;
}

}  // namespace

}  // extern "C"
namespace zc {
void debug_counts_decode(uint32_t out[2])
{
    dec_debug_counts_bf16(out);
    dec_debug_counts_fp8(out);
    dec_debug_counts_scale(out);
    dec_debug_counts_fp4(out);
}
}  // namespace zc
extern "C" {

uint32_t zc_test_decoder_warps(const zc_plan_t* p, uint32_t both_coded)
{
    DecShape sh;
    if (!p || dec_shape(p, both_coded != 0, &sh) != ZC_OK) return 0;
    return sh.warps;
}

zc_status zc_decompress(const zc_plan_t* p, const void* d_comp, size_t comp_bytes, void* d_out, void* d_workspace,
                        void* cuda_stream)
{
    return zc_decompress_xor(p, d_comp, comp_bytes, nullptr, d_out, d_workspace, cuda_stream);
}

zc_status zc_decompress_xor(const zc_plan_t* p, const void* d_comp, size_t comp_bytes, const void* d_base, void* d_out,
                            void* d_workspace, void* cuda_stream)
{
    if (d_base) {                                            // the delta form lives in the batched kernel
        if (!p) return ZC_E_INVALID_ARG;
        void* out1 = d_out;
        return zc_decompress_batch_xor(1, &p, &d_comp, &comp_bytes, &d_base, &out1, d_workspace, cuda_stream);
    }
    if (!p) return ZC_E_INVALID_ARG;
    return zc_decompress_chunks(p, d_comp, comp_bytes, 0, p->n_chunks, d_out, d_workspace, cuda_stream);
}

zc_status zc_decompress_chunks(const zc_plan_t* p, const void* d_comp, size_t comp_bytes, uint32_t first_chunk, uint32_t n_chunks,
                               void* d_out, void* d_workspace, void* cuda_stream)
{
    if (!p || !d_comp || !d_workspace || (!d_out && p->n_elems)) return ZC_E_INVALID_ARG;
    if ((uint64_t)first_chunk + n_chunks > p->n_chunks) return ZC_E_INVALID_ARG;
    if (!aligned16(d_comp) || !aligned16(d_out) || !aligned16(d_workspace)) return ZC_E_INVALID_ARG;
    if (comp_bytes < kHeaderBytes) return ZC_E_CORRUPT;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    DecShape shape;
    const zc_status ss = dec_shape(p, false, &shape);
    if (ss != ZC_OK) return ss;
    DecParams P{};
    P.comp = (const uint8_t*)d_comp;
    P.base = nullptr;
    // the kernel addresses the output by position in the tensor: d_out is where chunk first_chunk goes
    P.out = (uint8_t*)d_out - (size_t)first_chunk * p->chunk_bytes;
    P.c_begin = first_chunk; P.c_end = first_chunk + n_chunks;
    P.ctl = (Control*)d_workspace;
    P.comp_bytes = comp_bytes; P.input_bytes = p->input_bytes; P.n_syms = p->n_syms; P.n_elems = p->n_elems;
    P.n_chunks = p->n_chunks; P.cs = p->syms_per_chunk; P.sub = p->syms_per_sub; P.chunk_bytes = p->chunk_bytes;
    P.format = p->format; P.group = p->group;
    P.call_id = new_call_id();
    P.spec = comp_bytes >= kHeaderBytes + table_section_bytes(p->n_chunks, p->chunk_bytes) ? 1u : 0u;
    P.pool_bytes = shape.pool_bytes;
    P.spin_limit = test_knobs().spin_limit; P.skip_copy = test_knobs().skip_copy; P.sliced = shape.sliced;
    const uint32_t warps = shape.warps, ppl = shape.ppl;
    const size_t smem = shape.smem;
    // at least one block even for an empty range: the header is still checked
    const uint32_t want = std::max<uint32_t>((n_chunks + warps - 1) / warps, 1);
    const uint32_t grid = std::min<uint32_t>(want, (uint32_t)sm_count());
    const DecRanges R{d_comp, comp_bytes, d_out,
                      (size_t)std::min<uint64_t>((uint64_t)n_chunks * p->chunk_bytes, p->input_bytes - (uint64_t)first_chunk * p->chunk_bytes),
                      d_workspace, sizeof(Control)};
    cudaError_t e;
    switch (p->format) {
    case ZC_FMT_BF16: e = dec_launch_single_bf16(ppl, grid, warps * 32, smem, st, P, R); break;
    case ZC_FMT_FP8_E4M3: case ZC_FMT_FP8_E5M2: e = dec_launch_single_fp8(ppl, grid, warps * 32, smem, st, P, R); break;
    case ZC_FMT_SCALE_U8: e = dec_launch_single_scale(ppl, grid, warps * 32, smem, st, P, R); break;
    default: e = dec_launch_single_fp4(ppl, grid, warps * 32, smem, st, P, R); break;
    }
    return e == cudaSuccess ? ZC_OK : ZC_E_CUDA;
}

zc_status zc_decompress_batch(uint32_t n_tensors, const zc_plan_t* const* plans, const void* const* d_comp,
                              const size_t* comp_bytes, void* const* d_out, void* d_workspace, void* cuda_stream)
{
    return zc_decompress_batch_xor(n_tensors, plans, d_comp, comp_bytes, nullptr, d_out, d_workspace, cuda_stream);
}

zc_status zc_decompress_batch_xor(uint32_t n_tensors, const zc_plan_t* const* plans, const void* const* d_comp,
                                  const size_t* comp_bytes, const void* const* d_base, void* const* d_out,
                                  void* d_workspace, void* cuda_stream)
{
    if (!d_workspace || !aligned16(d_workspace)) return ZC_E_INVALID_ARG;
    if (n_tensors == 0) return ZC_OK;
    if (!plans || !d_comp || !comp_bytes || !d_out) return ZC_E_INVALID_ARG;
    for (uint32_t t = 0; t < n_tensors; ++t) {
        const zc_plan_t* p = plans[t];
        if (!p || !d_comp[t] || (!d_out[t] && p->n_elems)) return ZC_E_INVALID_ARG;
        if (!aligned16(d_comp[t]) || !aligned16(d_out[t]) || (d_base && !aligned16(d_base[t]))) return ZC_E_INVALID_ARG;
        if (p->format != plans[0]->format || p->chunk_bytes != plans[0]->chunk_bytes) return ZC_E_INVALID_ARG;
        if (comp_bytes[t] < kHeaderBytes) return ZC_E_CORRUPT;
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const zc_plan_t* p0 = plans[0];
    DecShape shape;
    bool delta = false;
    if (d_base) for (uint32_t t = 0; t < n_tensors; ++t) delta = delta || d_base[t] != nullptr;
    const zc_status ss = dec_shape(p0, delta, &shape);
    if (ss != ZC_OK) return ss;
    const unsigned long long call_id = new_call_id();
    static thread_local DecBatchParams B;                    // 28 KiB: kept off the stack
    for (uint32_t base = 0; base < n_tensors;) {
        B.ctl = (Control*)d_workspace;
        B.call_id = call_id;
        B.cs = p0->syms_per_chunk; B.sub = p0->syms_per_sub; B.chunk_bytes = p0->chunk_bytes;
        B.format = p0->format; B.group = p0->group; B.pool_bytes = shape.pool_bytes;
        B.tensor_base = base;
        B.spin_limit = test_knobs().spin_limit; B.skip_copy = test_knobs().skip_copy; B.sliced = shape.sliced;
        uint32_t n = 0;
        uint64_t total = 0;
        // as many tensors as fit one launch: at most kDecBatchMax, fewer than 2^32 chunks together
        while (base + n < n_tensors && n < kDecBatchMax && total + plans[base + n]->n_chunks < (1ull << 32)) {
            const zc_plan_t* p = plans[base + n];
            DecItem& it = B.item[n];
            it.comp = (const uint8_t*)d_comp[base + n];
            it.base = d_base ? (const uint8_t*)d_base[base + n] : nullptr;
            it.out = (uint8_t*)d_out[base + n];
            it.comp_bytes = comp_bytes[base + n]; it.input_bytes = p->input_bytes; it.n_syms = p->n_syms; it.n_elems = p->n_elems;
            it.n_chunks = p->n_chunks; it.first_chunk = (uint32_t)total;
            total += p->n_chunks;
            ++n;
        }
        B.n_tensors = n; B.total_chunks = (uint32_t)total;
        uint32_t with_chunks = 0;
        for (uint32_t i = 0; i < n; ++i) with_chunks += B.item[i].n_chunks != 0;
        // enough blocks for one chunk per warp, and (many small tensors, say the K/V pages of a step) for one
        // tensor per block, so that their tables are built side by side
        const uint32_t want = std::max<uint32_t>({(uint32_t)((total + shape.warps - 1) / shape.warps), with_chunks, 1u});
        const uint32_t grid = std::min<uint32_t>(want, (uint32_t)sm_count());
        // up to 8 ranges per block, none shorter than 16 chunks per warp (a range costs a table build); with fewer
        // tensors than blocks, one range per tensor at least
        B.n_ranges = grid * (uint32_t)std::min<uint64_t>(8, std::max<uint64_t>(1, total / ((uint64_t)grid * shape.warps * 16)));
        if (with_chunks <= grid) B.n_ranges = std::max<uint32_t>(B.n_ranges, with_chunks);
        B.n_ranges = (uint32_t)std::max<uint64_t>(1, std::min<uint64_t>(B.n_ranges, total));
        // the ranges are handed out through the ticket word of the control block
        if (cudaMemsetAsync(&B.ctl->ticket, 0, sizeof(uint32_t), st) != cudaSuccess) return ZC_E_CUDA;
        bool any_base = false;
        for (uint32_t i = 0; i < n; ++i) any_base = any_base || B.item[i].base != nullptr;
        DecRanges R{nullptr, 0, nullptr, 0, d_workspace, sizeof(Control)};
#if ZC_DEBUG_CHECKS
        DbgHull rd, wr;
        for (uint32_t i = 0; i < n; ++i) {
            rd.add(B.item[i].comp, B.item[i].comp_bytes);
            rd.add(B.item[i].base, B.item[i].input_bytes);
            wr.add(B.item[i].out, B.item[i].input_bytes);
        }
        R.in = rd.ptr(); R.in_bytes = rd.bytes(); R.out = wr.ptr(); R.out_bytes = wr.bytes();
#endif
        cudaError_t e;
        switch (p0->format) {
        case ZC_FMT_BF16: e = dec_launch_batch_bf16(shape.ppl, any_base, grid, shape.warps * 32, shape.smem, st, B, R); break;
        case ZC_FMT_FP8_E4M3: case ZC_FMT_FP8_E5M2: e = dec_launch_batch_fp8(shape.ppl, any_base, grid, shape.warps * 32, shape.smem, st, B, R); break;
        case ZC_FMT_SCALE_U8: e = dec_launch_batch_scale(shape.ppl, any_base, grid, shape.warps * 32, shape.smem, st, B, R); break;
        default: e = dec_launch_batch_fp4(shape.ppl, any_base, grid, shape.warps * 32, shape.smem, st, B, R); break;
        }
        if (e != cudaSuccess) return ZC_E_CUDA;
        base += n;
    }
    return ZC_OK;
}

zc_status zc_batch_status(const void* d_workspace, uint32_t* h_failed_tensor, void* cuda_stream)
{
    if (!d_workspace) return ZC_E_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    Control h;
    if (cudaMemcpyAsync(&h, d_workspace, sizeof(Control), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZC_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZC_E_CUDA;
    const bool mine = (h.status >> 8) == h.call_id && (h.status & 0xFF) != 0;
    if (h_failed_tensor) *h_failed_tensor = mine && h.failed ? h.failed - 1 : 0xFFFFFFFFu;
    return mine ? (zc_status)(h.status & 0xFF) : ZC_OK;
}

}  // extern "C"

#endif  // ZC_DEC_PART <= 1
