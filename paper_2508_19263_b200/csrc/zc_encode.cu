// Encoder kernel (split, bit packing, placement of the chunks by a look-back scan) and zc_compress,
// zc_compress_batch, zc_compress_noalloc, zc_device_status.
#include "zc_device.cuh"

#include <atomic>
#include <cstring>
#include <unordered_map>
#include <vector>

namespace zc {

// ------------------------------------------------------------------------------------------------
// parameters
// ------------------------------------------------------------------------------------------------

// Per symbol: the code left-aligned in bits 31..20 and its length in bits 3..0; a symbol without a code is 16.
struct EncTables { uint32_t enc[2][256]; };

// One tensor of a launch.
struct EncItem {
    const uint8_t* in;
    const uint8_t* base;                         // XOR-delta form: what is coded is in XOR base; or null
    uint8_t* out;
    uint64_t input_bytes, n_syms, n_elems;
    uint32_t n_chunks;
    uint32_t first_batch;                        // batches of all earlier tensors of the launch
    uint32_t index;                              // position in the caller's arrays (counters, error reports)
    uint32_t table;                              // its code tables among the uploaded ones (tensors may share a codebook)
    Layout lay;
};

// A launch covers N_ITEMS tensors at most (1: zc_compress, its table travels in the parameters;
// kEncBatchMax: zc_compress_batch, tables in global memory).  All tensors of a launch share format, chunk
// size and the modes of the two streams.
constexpr uint32_t kEncBatchMax = 256;           // keeps the parameter block below 32 KiB

struct EncCommon {
    Control* ctl;
    TensorCounters* counters;                    // indexed by EncItem::index
    unsigned long long* flags;                   // one look-back word per batch of the launch
    const EncTables* tables;                     // indexed by EncItem::index (batched launches)
    uint32_t cs, sub, chunk_bytes;               // symbols per chunk / per subchunk
    uint32_t format, group;
    uint32_t mode[2];
    uint32_t stage_stride;                       // bytes of one coded stream's lane regions per warp
    uint32_t region_bytes;                       // one lane region: n_slots * slot_bytes + sub + 4
    uint32_t slot_bytes;                         // one pack slot: sub (8 bits per symbol) or 1.5 * sub (12 bits)
    uint32_t sub_width;                          // bytes per sub_end entry (2 or 4)
    uint32_t n_slots;                            // pack slots per lane region (1..3, see encode_kernel)
    uint32_t sub_magic;                          // ceil(2^32 / sub): k / sub == umulhi(k, sub_magic) for k < 2^17
    uint32_t stage_step;                         // staging offset between a lane's consecutive groups (256 symbols apart)
                                                 // when that is a constant, i.e. sub divides 256; else 0
    uint32_t n_tensors, total_batches;
    uint32_t spin_limit;                         // polls after which a bounded wait gives up
};

template <int N_ITEMS> struct EncParamsT;
template <> struct EncParamsT<1> {
    EncCommon c;
    EncTables table;
    EncItem item[1];
};
template <> struct EncParamsT<(int)kEncBatchMax> {
    EncCommon c;
    EncItem item[kEncBatchMax];
};
static_assert(sizeof(EncParamsT<(int)kEncBatchMax>) < 32764, "kernel parameters are limited to 32764 bytes");

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

// Per-warp shared memory of one coded stream: 32 lane regions (+4 bytes of padding each, which also makes
// the region stride an odd number of words so that lanes walking their regions hit different banks).
// A region is n_slots pack slots of slot_bytes each, followed by the sub symbols of the lane's subchunk,
//   [pack 0 | .. | pack n_slots-1 | symbols].
// A lane packs the codes of its subchunk into pack slot (batch index mod n_slots), so the packed bits of the
// last n_slots batches are alive at the same time and the copy-out of a batch can wait up to n_slots
// iterations for the batch's position in the payload area (which comes from a look-back over other blocks).
// Two slot sizes:
//   slot_bytes = 1.5 * sub  holds any subchunk (codes are at most 12 bits).
//   slot_bytes = sub        holds 8 bits per symbol, which is plenty for streams that compress well and leaves
//                           room for one more slot.  Packing into the last slot may still run on into the
//                           symbols behind it (after k symbols at most 1.5 k bytes are written while the read
//                           position is sub + k, so the writer never passes unread symbols); packing into any
//                           other slot stops at the slot's end.  A chunk in which some lane needs more than its
//                           slot is finished on a slow path (everything older is copied out, then the chunk is
//                           packed again from slot 0 with the rest of the region as room) before anything else
//                           is staged.  That path waits for the chunk's own look-back, so the host picks this
//                           size only for code tables whose expected code length is well below 8 bits.

__device__ __forceinline__ void sts32_if(bool p, uint32_t addr, uint32_t v)
{
    if (p) ZC_DBG_SHARED(addr, 4, return);
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\t@q st.shared.u32 [%0], %1;\n\t}"
                 :: "r"(addr), "r"(v), "r"((uint32_t)p) : "memory");
}

// Append `len` bits (given left-aligned in `code`, zero below them) to a lane's bit accumulator and write a
// full 32-bit word to the region when one is complete and lies below `limit`.  hi holds the nb (< 32)
// pending bits left-aligned.
__device__ __forceinline__ void put_bits(uint32_t code, uint32_t len, uint32_t& hi, uint32_t& nb, uint32_t& waddr, uint32_t limit)
{
    if (nb + len > 31 && waddr < limit) ZC_DBG_SHARED(waddr, 4, return);
    hi |= code >> nb;
    const uint32_t lo = __funnelshift_r(0, code, nb);           // the bits that do not fit: code << (32 - nb), 0 if nb == 0
    const uint32_t n = nb + len;
    const bool full = n >= 32;
    // store if (n > 31 && waddr < limit): both compares and the store in one piece, so that the predicate never
    // travels through a register
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.gt.u32 p, %2, 31;\n\tsetp.lt.and.u32 q, %0, %3, p;\n\t@q st.shared.u32 [%0], %1;\n\t}"
                 :: "r"(waddr), "r"(hi), "r"(n), "r"(limit) : "memory");
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

// Writes the 128-byte header and the guard of one tensor; called by one thread once every chunk is in place.
__device__ void write_header(const EncCommon& C, const EncItem& I, TensorCounters* tc)
{
    const bool any_huff = C.mode[0] == ZC_MODE_HUFF || C.mode[1] == ZC_MODE_HUFF;
    const uint64_t payload_bytes = any_huff ? 16ull * ld_ctl(&tc->total16) : 0;
    uint8_t* h = I.out;
    uint32_t* h32 = reinterpret_cast<uint32_t*>(h);
    unsigned long long* h64 = reinterpret_cast<unsigned long long*>(h);
    for (int i = 0; i < 32; ++i) h32[i] = 0;
    h32[0] = kMagic;
    h[kHdrVersion] = 1; h[kHdrFormat] = (uint8_t)C.format; h[kHdrStreams] = 2;
    h64[kHdrElems / 8] = I.n_elems;
    h32[kHdrChunkBytes / 4] = C.chunk_bytes;
    h32[kHdrChunks / 4] = I.n_chunks;
    h[kHdrLmax] = kLmax; h[kHdrGroup] = (uint8_t)C.group; h[kHdrSubs] = kSubs; h[kHdrSubWidth] = (uint8_t)C.sub_width;
    const uint64_t total = I.lay.payload_off + payload_bytes + (any_huff ? 16 : 0);
    h64[kHdrTotal / 8] = total;
    h64[kHdrPayloadOff / 8] = I.lay.payload_off;
    h64[kHdrPayloadBytes / 8] = payload_bytes;
    for (int s = 0; s < 2; ++s) {
        uint8_t* d = h + kHdrStream0 + kHdrStreamStride * s;
        d[kSdMode] = (uint8_t)C.mode[s];
        reinterpret_cast<unsigned long long*>(d)[1] = I.n_syms;
        reinterpret_cast<unsigned long long*>(d)[2] = C.mode[s] == ZC_MODE_HUFF ? ld_ctl(&tc->payload_bits[s]) : 8 * I.n_syms;
        reinterpret_cast<unsigned long long*>(d)[3] = I.lay.section_off[s];
    }
    if (any_huff) {                              // 16 zero bytes behind the payload: decoders may peek past the last piece
        uint32_t* g = reinterpret_cast<uint32_t*>(I.out + I.lay.payload_off + payload_bytes);
        g[0] = g[1] = g[2] = g[3] = 0;
    }
    tc->total16 = total;                         // the host reads the container size from here
}

constexpr uint32_t kEncMaxWorkers = 8;       // worker warps per block = chunks per batch; one more warp hands out
                                             // the batches and places them
constexpr uint32_t kRing = 8;                // batches of a block whose bookkeeping is alive at the same time
constexpr uint32_t kTabSlots = 4;            // code tables (of the tensors the last batches belong to) alive at the same time
constexpr uint32_t kNoTensor = 0xFFFFFFFFu;  // "no more batches"
constexpr uint32_t kNoChunk = 0xFFFFFFFFu;
constexpr int kLookWide = 1;                 // look-back rounds cover 32 * kLookWide predecessors

// What a worker warp keeps about a chunk between packing it and copying it out.
struct PackedChunk {
    uint32_t c;                 // chunk index inside its tensor; kNoChunk: this warp had no chunk in the batch
    uint32_t t;                 // tensor (index into the launch's items)
    uint32_t end[2];            // per stream: inclusive scan of the subchunks' bit counts over the lanes (= sub_end)
};

// Whether the n staged symbols of every lane (at shared address src) all equal `symbol`; the whole warp calls it.
// Rarely needed (chunks that might be constant), so it is kept out of line.
__device__ __noinline__ bool all_symbols_are(uint32_t src, uint32_t n, uint32_t symbol)
{
    const uint32_t want = symbol * 0x01010101u;
    bool same = true;
    for (uint32_t i = 0; i < n / 4; ++i) same = same && lds32(src + 4 * i) == want;
    if (n & 3u) same = same && ((lds32(src + (n & ~3u)) ^ want) & (0xFFFFFFFFu >> (32 - 8 * (n & 3u)))) == 0;
    return __all_sync(0xFFFFFFFFu, same);
}

// The kernel.  A block is up to kEncMaxWorkers worker warps plus one service warp.
//
// Batches: the chunks of every tensor are grouped into batches of n_workers consecutive chunks, the batches of
// all tensors of the launch are numbered consecutively, and a global ticket counter hands them out in that
// order.  Worker w of the block that owns a batch encodes chunk w of it:
//   A  coalesced load, field split, raw stream stored as it is, coded stream staged per subchunk
//   B  every lane packs the codes of its subchunk into a pack slot of its lane region
//   C  subchunk end bits (sub_end table), the chunk's size in 16-byte units
//   D  (up to n_slots batches later) copy-out: every lane moves its bits to their place in the payload area
// The place of a chunk is the sum of the sizes of all earlier chunks of its tensor: the service warp adds up
// its block's batch and finds the rest with a decoupled look-back over the words other blocks publish.
//
// Worker 0 takes the ticket of batch i + 1 after packing batch i (as late as possible: batches must start in
// the order they were handed out, or the look-back of other blocks waits for a batch that is not even begun;
// measured, an earlier ticket costs more in look-back waits than it saves).  Part of the ticket's latency
// hides behind phase C; after it, if the ticket is another batch of the same tensor, worker 0 hands the batch
// out itself; otherwise it leaves the ticket to the service warp.
// The service warp never blocks on one thing: in a loop it (1) advances the look-back of the oldest unplaced
// batch by one round; (2) turns a ticket left to it into a batch: finds the tensor, copies the tensor's code
// table into a table slot and, for the first batch of a tensor, writes the fixed parts of the container.
// The warps are coupled only through words in shared memory (no block barrier in the loop):
//   s_ticket[i & 7], s_ticket_seq                  ticket of batch i; seq = tickets taken so far
//   s_tensor/s_cbase/s_tabslot[i & 7], s_base_seq  batch i of this block; seq = batches handed out so far
//   s_tot[i & 7][w], s_cnt[i & 7]                  size of worker w's chunk; cnt = workers that posted it
//   s_off[i & 7][w], s_off_seq                     position of that chunk; seq = batches placed so far
// A worker has copied out batch i - n_slots (n_slots <= 3) before it packs batch i; a batch is placed only
// after every worker has posted its size, so worker 0 never hands out a batch more than 3 ahead of the last
// placed one, and the service warp hands one out only while fewer than 4 are unplaced.  So all warps of a
// block are within 4 batches of each other and rings of 8 are enough.  A table slot is reused only when every worker has posted the last batch that used it.
// H0 / H1: stream 0 / 1 is Huffman-coded (the same for every tensor of a launch; a template parameter so that
// the code of a raw stream's packing and copy-out does not exist and the kernel stays small).
template <int FMT, int N_ITEMS, bool H0, bool H1>
// (with both streams coded the lane regions leave room for two blocks per SM at most: those kernels may use the registers of a third)
__global__ void __launch_bounds__((kEncMaxWorkers + 1) * 32, (H0 && H1) ? 2 : 3)
encode_kernel(const __grid_constant__ EncParamsT<N_ITEMS> P)
{
    extern __shared__ __align__(16) uint8_t smem[];
    const EncCommon& C = P.c;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n_workers = (blockDim.x >> 5) - 1;
    const bool service = warp == n_workers;
    constexpr uint32_t n_huff = (H0 ? 1u : 0u) + (H1 ? 1u : 0u);
    auto is_huff = [](const int s) constexpr { return s == 0 ? H0 : H1; };
    const uint32_t n_slots = C.n_slots;

    // shared: tables[kTabSlots][n_huff][256] | per worker warp: regions[n_huff][stage_stride]
    uint32_t* tabs = reinterpret_cast<uint32_t*>(smem);
    const uint32_t tab_words = 256 * (n_huff ? n_huff : 1);     // words of one table slot
    uint8_t* stage = smem + 4 * kTabSlots * tab_words + (size_t)(service ? 0 : warp) * n_huff * C.stage_stride;
    const uint32_t region = C.region_bytes;                     // n_slots * slot_bytes + sub + 4
    const uint32_t sym_off = n_slots * C.slot_bytes;            // symbols sit at this offset inside a region

    __shared__ uint32_t s_ticket[kRing], s_tensor[kRing], s_cbase[kRing], s_tabslot[kRing], s_cnt[kRing];
    __shared__ uint32_t s_ticket_seq, s_base_seq, s_off_seq, s_fail;
    __shared__ uint32_t s_fill[kTabSlots][2];                   // per table slot and coded stream: fill symbol | its code length << 8
    __shared__ unsigned long long s_tot[kRing][kEncMaxWorkers], s_off[kRing][kEncMaxWorkers];

    if (threadIdx.x < kRing) s_cnt[threadIdx.x] = 0;
    if (threadIdx.x == 0) {
        s_fail = 0; s_off_seq = 0; s_base_seq = 0;
        s_ticket[0] = atomicAdd(&C.ctl->ticket, 1u);
        s_ticket_seq = 1;
    }
    __syncthreads();

    auto vol32 = [](const uint32_t* p) { return *reinterpret_cast<const volatile uint32_t*>(p); };
    auto item = [&](const uint32_t t) -> const EncItem& { return P.item[N_ITEMS == 1 ? 0u : t]; };
    auto counters = [&](const uint32_t t) -> TensorCounters* { return C.counters + (N_ITEMS == 1 ? 0u : P.item[t].index); };

    if (service) {
        // =========================== the service warp ===========================
        // block 0: tensors without chunks are all header
        if (blockIdx.x == 0 && lane == 0)
            for (uint32_t t = 0; t < C.n_tensors; ++t)
                if (item(t).n_chunks == 0) write_header(C, item(t), counters(t));

        uint32_t handed = 0, placed = 0;                         // batches of this block handed out / placed
        uint32_t tcur = 0;                                       // tensor of the last ticket (tickets only grow)
        uint32_t tab_tensor = kNoTensor, tab_slot = 0;           // the newest table slot and whose table it holds
        uint32_t slot_last0 = 0, slot_last1 = 0, slot_last2 = 0, slot_last3 = 0;   // 1 + last batch that used slot k
        bool ended = false, lb_on = false;
        unsigned long long lb_sum = 0, lb_own = 0, lb_inc = 0, lb_v = 0;
        long long lb_base = 0;
        unsigned long long* lb_flags = nullptr;
        uint32_t lb_b = 0, idle = 0;
        // Loads tensor t's code tables into the slot after the newest one, once every worker has posted the last
        // batch that was packed with the table that is there now; false when that is not yet the case.
        auto load_next_slot = [&](const uint32_t t, const uint32_t placed_now) -> bool {
            const uint32_t nslot = (tab_slot + 1) % kTabSlots;
            const uint32_t last = nslot == 0 ? slot_last0 : nslot == 1 ? slot_last1 : nslot == 2 ? slot_last2 : slot_last3;
            if (placed_now < last) return false;
            uint32_t* tab = tabs + nslot * tab_words;
            uint32_t hs = 0;
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                if (!is_huff(s)) continue;
                const uint32_t* src;
                if constexpr (N_ITEMS == 1) src = P.table.enc[s]; else src = C.tables[item(t).table].enc[s];
                // the fill symbol (needed when both streams are coded) is the one whose code is all zeros: its
                // entry is nothing but its length
                uint32_t fill = 0xFFFFFFFFu;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const uint32_t v = src[lane + 32 * i];
                    tab[256 * hs + lane + 32 * i] = v;
                    if (v >= 1 && v <= kLmax) fill = (lane + 32 * i) | (v << 8);
                }
                {
                    const uint32_t who = __ballot_sync(0xFFFFFFFFu, fill != 0xFFFFFFFFu);
                    fill = __shfl_sync(0xFFFFFFFFu, fill, who ? __ffs(who) - 1 : 0);
                    if (lane == 0) s_fill[nslot][hs] = who ? fill : 0xFF00u;     // no code at all: a length no chunk can match
                }
                ++hs;
            }
            __syncwarp();
            return true;
        };
        for (;;) {
            bool did = false;
            // batches worker 0 handed out itself since the last look: they use the newest table slot
            const uint32_t tickets = vol32(&s_ticket_seq);       // read before s_base_seq (worker 0 writes it after)
            __threadfence_block();
            const uint32_t published = vol32(&s_base_seq);
            if (published > handed) {
                handed = published;
                if (tab_slot == 0) slot_last0 = handed; else if (tab_slot == 1) slot_last1 = handed;
                else if (tab_slot == 2) slot_last2 = handed; else slot_last3 = handed;
            }
            // ---- (1) placement of the oldest unplaced batch ----
            const uint32_t real = ended ? handed - 1 : handed;   // the last ticket was "no more batches"
            if (placed < real) {
                const uint32_t r = placed % kRing;
                if (!lb_on && vol32(&s_cnt[r]) == n_workers) {   // every worker has posted a size (0 without a chunk)
                    __threadfence_block();
                    if (lane == 0) s_cnt[r] = 0;
                    lb_v = lane < n_workers ? *reinterpret_cast<const volatile unsigned long long*>(&s_tot[r][lane]) : 0ull;
                    lb_inc = lb_v;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const unsigned long long x = __shfl_up_sync(0xFFFFFFFFu, lb_inc, o);
                        if (lane >= (uint32_t)o) lb_inc += x;
                    }
                    lb_own = __shfl_sync(0xFFFFFFFFu, lb_inc, 31);
                    const EncItem& I = item(vol32(&s_tensor[r]));
                    lb_flags = C.flags + I.first_batch;          // the look-back stays inside the tensor
                    lb_b = vol32(&s_ticket[r]) - I.first_batch;
                    lb_sum = 0;
                    lb_base = (long long)lb_b - 1;               // lane i looks at batch lb_base - i
                    if (n_huff && lb_b != 0 && lane == 0) st_flag(&lb_flags[lb_b], kFlagAggregate | lb_own);
                    lb_on = true;
                    did = true;
                }
                if (lb_on) {
                    bool done = !n_huff || lb_b == 0;
                    if (!done) {
                        // One round of the look-back: kLookWide * 32 predecessors at a time, newest first, up to the
                        // first one that already knows its prefix.  All loads of a round are in flight together, so a
                        // round costs one trip to the L2 however wide it is; it has to be wider than the number of
                        // batches in flight (one per resident block), or the prefixes of a turn form a chain of
                        // rounds from block to block.
                        unsigned long long f[kLookWide];
#pragma unroll
                        for (int k = 0; k < kLookWide; ++k) {
                            const long long idx = lb_base - 32 * k - lane;
                            f[k] = idx >= 0 ? ld_flag(&lb_flags[idx]) : kFlagPrefix;      // before batch 0: prefix 0
                        }
                        unsigned long long x = 0;
                        bool found = false, stuck = false;
#pragma unroll
                        for (int k = 0; k < kLookWide; ++k) {
                            if (found || stuck) continue;
                            const uint32_t ready = __ballot_sync(0xFFFFFFFFu, (f[k] >> 62) != 0);
                            const uint32_t prefix = __ballot_sync(0xFFFFFFFFu, (f[k] >> 62) == 2);
                            const uint32_t first_prefix = prefix ? (uint32_t)__ffs(prefix) - 1 : 32u;
                            const uint32_t need = first_prefix == 32 ? 0xFFFFFFFFu : (0xFFFFFFFFu >> (31 - first_prefix));
                            if ((ready & need) != need) { stuck = true; continue; }
                            if (lane <= first_prefix || first_prefix == 32) x += f[k] & kFlagValue;
                            found = first_prefix != 32;
                        }
                        if (!stuck) {
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
                            lb_sum += x;
                            if (found) done = true; else lb_base -= 32 * kLookWide;
                            did = true;
                        }
                    }
                    if (done) {
                        if (n_huff && lane == 0) st_flag(&lb_flags[lb_b], kFlagPrefix | (lb_sum + lb_own));
                        if (lane < n_workers) s_off[r][lane] = lb_sum + lb_inc - lb_v;
                        __threadfence_block();
                        __syncwarp();
                        if (lane == 0) *reinterpret_cast<volatile uint32_t*>(&s_off_seq) = placed + 1;
                        ++placed;
                        lb_on = false;
                        did = true;
                    }
                }
            }
            // ---- (2) a new ticket becomes a batch ----
            if (!ended && handed < tickets && handed < placed + 4) {
                const uint32_t g = vol32(&s_ticket[handed % kRing]);
                uint32_t t = kNoTensor, cbase = 0;
                bool publish = true;
                if (g < C.total_batches) {
                    if (N_ITEMS > 1)                             // tensors without chunks share their start with the next one
                        while (tcur + 1 < C.n_tensors && g >= P.item[tcur + 1].first_batch) ++tcur;
                    t = tcur;
                    const EncItem& I = item(t);
                    cbase = (g - I.first_batch) * n_workers;
                    if (n_huff && t != tab_tensor) {
                        // another tensor: its table goes to the next slot
                        if (load_next_slot(t, placed + (lb_on ? 1u : 0u))) {
                            tab_slot = (tab_slot + 1) % kTabSlots;
                            tab_tensor = t;
                        } else {
                            publish = false;                     // not yet: look back some more first
                        }
                    }
                    if (publish && g == I.first_batch) {
                        // the fixed parts of the tensor's container: code lengths, padding of the chunk offset
                        // table, tail padding of raw bodies
                        const uint32_t* tab = tabs + tab_slot * tab_words;
                        uint32_t hs = 0;
#pragma unroll
                        for (int s = 0; s < 2; ++s) {
                            if (is_huff(s)) {
                                for (uint32_t v = lane; v < 256; v += 32) I.out[I.lay.section_off[s] + v] = (uint8_t)(tab[256 * hs + v] & 15);
                                const uint32_t padded = (I.n_chunks + 3) & ~3u;
                                for (uint32_t i = I.n_chunks + lane; i < padded; i += 32)
                                    reinterpret_cast<uint32_t*>(I.out + I.lay.chunk_off_tab[s])[i] = 0;
                                ++hs;
                            } else {
                                const uint64_t lo = (I.n_syms + 7) & ~7ull, hi = (I.n_syms + 15) & ~15ull;
                                for (uint64_t i = lo + lane; i < hi; i += 32) I.out[I.lay.section_off[s] + i] = 0;
                            }
                        }
                    }
                } else {
                    ended = true;
                }
                if (publish) {
                    if (t != kNoTensor) {
                        if (tab_slot == 0) slot_last0 = handed + 1; else if (tab_slot == 1) slot_last1 = handed + 1;
                        else if (tab_slot == 2) slot_last2 = handed + 1; else slot_last3 = handed + 1;
                    }
                    __syncwarp();
                    if (lane == 0) {
                        s_tensor[handed % kRing] = t; s_cbase[handed % kRing] = cbase; s_tabslot[handed % kRing] = tab_slot;
                        __threadfence_block();
                        *reinterpret_cast<volatile uint32_t*>(&s_base_seq) = handed + 1;
                    }
                    ++handed;
                    did = true;
                }
            }
            if (ended && placed == handed - 1) break;
            if (vol32(&s_fail)) break;
            if (did) { idle = 0; continue; }
            if (++idle > C.spin_limit) { s_fail = 1; break; }
            __nanosleep(1000);                                   // nothing to do right now: leave the issue slots to the workers
        }
    } else {
        // =========================== a worker warp ===========================
        // Bounded wait of the whole warp until a sequence word reaches `target`; false on a failure flag or
        // when the wait gives up.
        auto wait_seq = [&](const uint32_t* word, const uint32_t target) -> bool {
            bool ok = false;
            for (uint32_t n = 0; n < C.spin_limit; ++n) {
                if (vol32(word) >= target) { ok = true; break; }
                if (vol32(&s_fail)) break;
                if (n > 64) __nanosleep(40);
            }
            __syncwarp();
            __threadfence_block();
            return ok;
        };

        // Chunks this warp has completely written, per tensor; added to the tensor's counter (behind a fence)
        // when the warp moves on to another tensor or leaves.  Whoever completes a tensor writes its header.
        uint32_t acc_t = kNoTensor, acc_n = 0;
        unsigned long long acc_bits0 = 0, acc_bits1 = 0;           // lane 0: payload bits of those chunks, per stream
        auto flush_acc = [&]() {
            if (acc_n == 0) return;
            __threadfence();
            __syncwarp();
            if (lane == 0) {
                TensorCounters* tc = counters(acc_t);
                if (H0) atomicAdd(&tc->payload_bits[0], acc_bits0);
                if (H1) atomicAdd(&tc->payload_bits[1], acc_bits1);
                __threadfence();
                const uint32_t before = atomicAdd(&tc->done, acc_n);
                if (before + acc_n == item(acc_t).n_chunks) {
                    __threadfence();
                    write_header(C, item(acc_t), tc);
                }
            }
            acc_n = 0;
            acc_bits0 = acc_bits1 = 0;
        };
        auto chunk_done = [&](const uint32_t t, const uint32_t bits0, const uint32_t bits1) {
            if (t != acc_t) { flush_acc(); acc_t = t; }
            ++acc_n;
            acc_bits0 += bits0; acc_bits1 += bits1;
        };

        // ---- copy-out of a packed chunk: every lane moves its bits to their final position in the piece ----
        auto copy_out = [&](const PackedChunk& pc, const uint32_t slot, const uint64_t off16) {
            const EncItem& I = item(pc.t);
            uint32_t hs = 0;
            uint64_t piece_off16 = off16;
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                if (!is_huff(s)) continue;
                const uint32_t end = pc.end[s];
                uint32_t start = __shfl_up_sync(0xFFFFFFFFu, end, 1);
                if (lane == 0) start = 0;
                const uint32_t bits = end - start;
                const uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, end, 31);
                const uint32_t piece16 = (chunk_bits + 127) / 128;
                if (lane == 0) reinterpret_cast<uint32_t*>(I.out + I.lay.chunk_off_tab[s])[pc.c] = (uint32_t)piece_off16;
                uint32_t* piece = reinterpret_cast<uint32_t*>(I.out + I.lay.payload_off + 16 * piece_off16);
                const uint32_t piece_words = 4 * piece16;
                const uint32_t reg_s = smem_u32(stage + hs * C.stage_stride + lane * region) + slot;
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
            if (lane == 0 && pc.c == I.n_chunks - 1) counters(pc.t)->total16 = piece_off16;
            __syncwarp();
            chunk_done(pc.t, H0 ? __shfl_sync(0xFFFFFFFFu, pc.end[0], 31) : 0u, H1 ? __shfl_sync(0xFFFFFFFFu, pc.end[1], 31) : 0u);
        };

        uint32_t bad = 0;                                           // 1 + tensor in which a symbol had no code
        // packed chunks that wait for their copy-out, newest first: q0 is batch it - 1, q1 batch it - 2, ...
        PackedChunk q0{kNoChunk, 0, {0, 0}}, q1 = q0, q2 = q0;
        uint32_t n_pend = 0;
        uint32_t slot_idx = 0;                                      // pack slot of batch `it`: it mod n_slots
        // waits until the oldest pending batch is placed and copies this warp's chunk of it out
        auto flush_oldest = [&](const uint32_t it) -> bool {
            const uint32_t j = it - n_pend;                         // the batch in question
            if (!wait_seq(&s_off_seq, j + 1)) return false;
            if (n_huff) {
                PackedChunk pc;
                pc.c = n_pend == 1 ? q0.c : n_pend == 2 ? q1.c : q2.c;
                pc.t = n_pend == 1 ? q0.t : n_pend == 2 ? q1.t : q2.t;
                pc.end[0] = n_pend == 1 ? q0.end[0] : n_pend == 2 ? q1.end[0] : q2.end[0];
                pc.end[1] = n_pend == 1 ? q0.end[1] : n_pend == 2 ? q1.end[1] : q2.end[1];
                // its slot: the slots are used round-robin, so it lies n_pend steps behind the current one
                const uint32_t sl = (slot_idx + n_slots * 4 - n_pend) % n_slots;
                if (pc.c != kNoChunk)
                    copy_out(pc, sl * C.slot_bytes, *reinterpret_cast<const volatile unsigned long long*>(&s_off[j % kRing][warp]));
            }
            --n_pend;
            return true;
        };
        bool failed = false;
        for (uint32_t it = 0;; ++it) {
            if (!wait_seq(&s_base_seq, it + 1)) { failed = true; break; }
            const uint32_t t = vol32(&s_tensor[it % kRing]);
            if (t == kNoTensor) {
                while (n_pend && !failed) failed = !flush_oldest(it);
                break;
            }
            const EncItem& I = item(t);
            const uint32_t my_c = vol32(&s_cbase[it % kRing]) + warp;
            const bool active = my_c < I.n_chunks;
            PackedChunk cur{active ? my_c : kNoChunk, t, {0, 0}};
            const uint32_t slot = slot_idx * C.slot_bytes;
            const uint64_t c_lo = (uint64_t)(active ? my_c : 0) * C.cs;
            const uint32_t c_syms = active ? (uint32_t)min((uint64_t)C.cs, I.n_syms - c_lo) : 0u;

            // ---- phase A: coalesced load, split, raw stream stored as is, coded stream staged per subchunk ----
            // Group g (16 input bytes = symbols 8 g .. 8 g + 7) is staged at byte (8 g / sub) * region + 8 g % sub of
            // the symbol area.  A lane's groups are 32 apart: when sub divides 256 that is a constant step.
            uint8_t* const raw0 = I.out + I.lay.section_off[0] + c_lo;      // this chunk in the raw bodies
            uint8_t* const raw1 = I.out + I.lay.section_off[1] + c_lo;
            const uint32_t sym_s = smem_u32(stage) + sym_off;
            const uint32_t step = C.stage_step;
            auto stage_off = [&](const uint32_t g_) {
                const uint32_t k = 8 * g_, j = __umulhi(k, C.sub_magic);
                return j * region + (k - j * C.sub);
            };
            // A complete chunk of nothing but a coded stream's fill symbol takes no bits and need not be packed.  With both
            // streams coded (delta checkpoints: stretches of unchanged weights are such chunks in both streams) every
            // staged word is compared with the fill symbol on the way, one logic operation per word; with one coded
            // stream such chunks are rare and are found after packing (phase C), so that path pays nothing here.
            constexpr bool kSpotConstant = H0 && H1;
            const uint32_t tab_slot_idx = vol32(&s_tabslot[it % kRing]);
            uint32_t fill4[2] = {0, 0}, differs[2] = {1, 1};
            if (kSpotConstant) {
#pragma unroll
                for (int hs = 0; hs < 2; ++hs) {
                    fill4[hs] = (vol32(&s_fill[tab_slot_idx][hs]) & 0xFFu) * 0x01010101u;
                    differs[hs] = 0;
                }
            }
            auto stage_group = [&](const uint4 x, const uint32_t g_, const uint32_t off) {
                const uint32_t w[4] = {x.x, x.y, x.z, x.w};
                uint32_t sy[2][2];
                split16<FMT>(w, sy[0], sy[1]);
                uint32_t hs = 0;
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    if (!is_huff(s)) {
                        st_cs_v2((s == 0 ? raw0 : raw1) + 8 * g_, make_uint2(sy[s][0], sy[s][1]));
                    } else {
                        sts32(sym_s + hs * C.stage_stride + off, sy[s][0]);
                        sts32(sym_s + hs * C.stage_stride + off + 4, sy[s][1]);
                        if (kSpotConstant) differs[hs] |= (sy[s][0] ^ fill4[hs]) | (sy[s][1] ^ fill4[hs]);
                        ++hs;
                    }
                }
            };
            const uint32_t n_vec = (c_syms + 7) / 8;
            const uint8_t* src_c = I.in + 2 * c_lo;
            uint32_t g = lane;
            uint32_t off = stage_off(lane);                             // running offset (constant-step case)
            auto off_at = [&](const uint32_t g_, const uint32_t i) { return step ? off + i * step : stage_off(g_); };
            if (I.base) {
                // delta form: the chunk of the base tensor is read alongside and XOR-ed in (two pairs of loads in flight)
                const uint8_t* base_c = I.base + 2 * c_lo;
                auto x4 = [](const uint4 a, const uint4 b) { return make_uint4(a.x ^ b.x, a.y ^ b.y, a.z ^ b.z, a.w ^ b.w); };
                if (2 * (c_lo + 8ull * n_vec) <= I.input_bytes) {
                    for (; g + 32 < n_vec; g += 64, off += 2 * step) {
                        const uint4 x0 = ld_nc_v4(src_c + 16 * g), y0 = ld_nc_v4(base_c + 16 * g);
                        const uint4 x1 = ld_nc_v4(src_c + 16 * (g + 32)), y1 = ld_nc_v4(base_c + 16 * (g + 32));
                        stage_group(x4(x0, y0), g, off_at(g, 0));
                        stage_group(x4(x1, y1), g + 32, off_at(g + 32, 1));
                    }
                    for (; g < n_vec; g += 32, off += step)
                        stage_group(x4(ld_nc_v4(src_c + 16 * g), ld_nc_v4(base_c + 16 * g)), g, off_at(g, 0));
                } else {
                    for (; g < n_vec; g += 32)
                        stage_group(x4(load16_guarded(I.in, 2 * (c_lo + 8ull * g), I.input_bytes),
                                       load16_guarded(I.base, 2 * (c_lo + 8ull * g), I.input_bytes)), g, stage_off(g));
                }
            } else if (2 * (c_lo + 8ull * n_vec) <= I.input_bytes) {    // every group of this chunk is complete
                for (; g + 96 < n_vec; g += 128, off += 4 * step) {         // four loads in flight per lane
                    const uint4 x0 = ld_nc_v4(src_c + 16 * g);
                    const uint4 x1 = ld_nc_v4(src_c + 16 * (g + 32));
                    const uint4 x2 = ld_nc_v4(src_c + 16 * (g + 64));
                    const uint4 x3 = ld_nc_v4(src_c + 16 * (g + 96));
                    stage_group(x0, g, off_at(g, 0));
                    stage_group(x1, g + 32, off_at(g + 32, 1));
                    stage_group(x2, g + 64, off_at(g + 64, 2));
                    stage_group(x3, g + 96, off_at(g + 96, 3));
                }
                for (; g < n_vec; g += 32, off += step) stage_group(ld_nc_v4(src_c + 16 * g), g, off_at(g, 0));
            } else {
                for (; g < n_vec; g += 32) stage_group(load16_guarded(I.in, 2 * (c_lo + 8ull * g), I.input_bytes), g, stage_off(g));
            }
            __syncwarp();

            // Warm the L2 for the batch one round of tickets ahead (whichever block gets it; it may lie in one of
            // the next tensors): the loads of phase A are the longest wait of a turn.  One 128-byte line per lane
            // and 4 KiB of chunk.
            {
                uint32_t g2 = vol32(&s_ticket[it % kRing]) + gridDim.x, t2 = t;
                if (N_ITEMS > 1)
                    for (uint32_t hop = 0; hop < 4 && t2 + 1 < C.n_tensors && g2 >= P.item[N_ITEMS > 1 ? t2 + 1 : 0].first_batch; ++hop) ++t2;
                const EncItem& I2 = item(t2);
                const uint64_t c2 = (uint64_t)(g2 - I2.first_batch) * n_workers + warp;
                if (g2 < C.total_batches && c2 < I2.n_chunks) {
                    const uint64_t lo = c2 * C.chunk_bytes;
                    for (uint32_t o = 128 * lane; o < C.chunk_bytes; o += 4096)
                        if (lo + o < I2.input_bytes) {
                            asm volatile("prefetch.global.L2 [%0];" :: "l"(I2.in + lo + o));
                            if (I2.base) asm volatile("prefetch.global.L2 [%0];" :: "l"(I2.base + lo + o));
                        }
                }
            }

            // the chunk that was packed into this slot n_slots batches ago must leave before this one is packed
            if (n_pend == n_slots && !flush_oldest(it)) { failed = true; break; }

            // ---- phase B: every lane packs the codes of its subchunk into its pack slot, from bit 0 ----
            const uint32_t lo_sym = lane * C.sub;
            const uint32_t n_my = lo_sym < c_syms ? min(C.sub, c_syms - lo_sym) : 0u;
            const uint32_t tab_slot_s = smem_u32(tabs + tab_slot_idx * tab_words);
            // batches below this ticket belong to the same tensor
            const uint32_t t_end = (N_ITEMS > 1 && t + 1 < C.n_tensors) ? P.item[N_ITEMS > 1 ? t + 1 : 0].first_batch : C.total_batches;
            // returns the bit count; stores stop at `room` bytes (the count goes on)
            auto pack = [&](const uint32_t hs, const uint32_t slot_off, const uint32_t room) -> uint32_t {
                const uint32_t reg_s = smem_u32(stage + hs * C.stage_stride + lane * region);
                const uint32_t tab_s = tab_slot_s + 1024 * hs;
                const uint32_t w0 = reg_s + slot_off, limit = w0 + room;
                uint32_t hi = 0, nb = 0, waddr = w0, seen = 0;
                const uint32_t src = reg_s + sym_off;
                const uint32_t full_words = n_my / 4;
                for (uint32_t i = 0; i < full_words; ++i) {
                    const uint32_t four = lds32(src + 4 * i);
                    // table index = one byte of the word (byte permute), scaled by 4 in the address add
                    const uint32_t e0 = lds32(tab_s + 4u * __byte_perm(four, 0, 0x4440));
                    const uint32_t e1 = lds32(tab_s + 4u * __byte_perm(four, 0, 0x4441));
                    const uint32_t e2 = lds32(tab_s + 4u * __byte_perm(four, 0, 0x4442));
                    const uint32_t e3 = lds32(tab_s + 4u * __byte_perm(four, 0, 0x4443));
                    seen |= e0 | e1 | e2 | e3;
                    // two codes at a time: the second one shifted behind the first (the funnel shift takes its
                    // count from the low 5 bits of the first entry = its length); the length fields end up below
                    // bit 8 and are masked off
                    const uint32_t ca = (e0 | __funnelshift_r(e1, 0, e0)) & 0xFFFFFF00u;
                    put_bits(ca, (e0 + e1) & 31, hi, nb, waddr, limit);
                    const uint32_t cb = (e2 | __funnelshift_r(e3, 0, e2)) & 0xFFFFFF00u;
                    put_bits(cb, (e2 + e3) & 31, hi, nb, waddr, limit);
                }
                for (uint32_t i = 4 * full_words; i < n_my; ++i) {      // ragged end of the last chunk
                    const uint32_t four = lds32(src + (i & ~3u));
                    const uint32_t e = lds32(tab_s + (((four >> (8 * (i & 3))) & 0xFF) << 2));
                    seen |= e;
                    put_bits(e & 0xFFFFFF00u, e & 31, hi, nb, waddr, limit);
                }
                if (active && waddr < limit) sts32(waddr, hi);          // pending bits (or zero)
                if (seen & 16) bad = t + 1;                             // an entry without a code carries bit 4
                return 8 * (waddr - w0) + nb;
            };
            // Both streams at once: two independent accumulators per lane, their table lookups and shifts issued
            // alternately (one stream's shared-memory latency is covered by the other's arithmetic).
            auto pack2 = [&](const uint32_t slot_off, const uint32_t room, uint32_t& bits_a, uint32_t& bits_b) {
                const uint32_t rega = smem_u32(stage + lane * region), regb = rega + C.stage_stride;
                const uint32_t taba = tab_slot_s, tabb = tab_slot_s + 1024;
                const uint32_t wa0 = rega + slot_off, lima = wa0 + room, wb0 = regb + slot_off, limb = wb0 + room;
                uint32_t hia = 0, nba = 0, wa = wa0, hib = 0, nbb = 0, wb = wb0, seen = 0;
                const uint32_t srca = rega + sym_off, srcb = regb + sym_off;
                const uint32_t full_words = n_my / 4;
                for (uint32_t i = 0; i < full_words; ++i) {
                    const uint32_t fa = lds32(srca + 4 * i), fb = lds32(srcb + 4 * i);
                    const uint32_t a0 = lds32(taba + 4u * __byte_perm(fa, 0, 0x4440));
                    const uint32_t b0 = lds32(tabb + 4u * __byte_perm(fb, 0, 0x4440));
                    const uint32_t a1 = lds32(taba + 4u * __byte_perm(fa, 0, 0x4441));
                    const uint32_t b1 = lds32(tabb + 4u * __byte_perm(fb, 0, 0x4441));
                    const uint32_t a2 = lds32(taba + 4u * __byte_perm(fa, 0, 0x4442));
                    const uint32_t b2 = lds32(tabb + 4u * __byte_perm(fb, 0, 0x4442));
                    const uint32_t a3 = lds32(taba + 4u * __byte_perm(fa, 0, 0x4443));
                    const uint32_t b3 = lds32(tabb + 4u * __byte_perm(fb, 0, 0x4443));
                    seen |= a0 | a1 | a2 | a3 | b0 | b1 | b2 | b3;
                    put_bits((a0 | __funnelshift_r(a1, 0, a0)) & 0xFFFFFF00u, (a0 + a1) & 31, hia, nba, wa, lima);
                    put_bits((b0 | __funnelshift_r(b1, 0, b0)) & 0xFFFFFF00u, (b0 + b1) & 31, hib, nbb, wb, limb);
                    put_bits((a2 | __funnelshift_r(a3, 0, a2)) & 0xFFFFFF00u, (a2 + a3) & 31, hia, nba, wa, lima);
                    put_bits((b2 | __funnelshift_r(b3, 0, b2)) & 0xFFFFFF00u, (b2 + b3) & 31, hib, nbb, wb, limb);
                }
                for (uint32_t i = 4 * full_words; i < n_my; ++i) {      // ragged end of the last chunk
                    const uint32_t fa = lds32(srca + (i & ~3u)), fb = lds32(srcb + (i & ~3u));
                    const uint32_t ea = lds32(taba + (((fa >> (8 * (i & 3))) & 0xFF) << 2));
                    const uint32_t eb = lds32(tabb + (((fb >> (8 * (i & 3))) & 0xFF) << 2));
                    seen |= ea | eb;
                    put_bits(ea & 0xFFFFFF00u, ea & 31, hia, nba, wa, lima);
                    put_bits(eb & 0xFFFFFF00u, eb & 31, hib, nbb, wb, limb);
                }
                if (active && wa < lima) sts32(wa, hia);
                if (active && wb < limb) sts32(wb, hib);
                if (seen & 16) bad = t + 1;
                bits_a = 8 * (wa - wa0) + nba;
                bits_b = 8 * (wb - wb0) + nbb;
            };
            bool oversize = false;
            uint32_t my_bits[2] = {0, 0};
            const bool last_slot = slot_idx + 1 == n_slots;
            bool packed_both = false;
            if (H0 && H1) {
                bool constant[2];
#pragma unroll
                for (int hs = 0; hs < 2; ++hs)
                    constant[hs] = kSpotConstant && __all_sync(0xFFFFFFFFu, differs[hs] == 0) && active && c_syms == C.cs &&
                                   (vol32(&s_fill[tab_slot_idx][hs]) >> 8) <= kLmax;
                if (!constant[0] && !constant[1]) {
                    pack2(slot, last_slot ? C.slot_bytes + C.sub : C.slot_bytes, my_bits[0], my_bits[1]);
                    oversize = my_bits[0] > 8 * C.slot_bytes || my_bits[1] > 8 * C.slot_bytes;
                    packed_both = true;
                }
            }
            if (!packed_both) {
                uint32_t hs = 0;
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    if (!is_huff(s)) continue;
                    // nothing but the fill symbol (which has a code): no bits, nothing to pack
                    const bool constant = kSpotConstant && __all_sync(0xFFFFFFFFu, differs[hs] == 0) && active &&
                                          c_syms == C.cs && (vol32(&s_fill[tab_slot_idx][hs]) >> 8) <= kLmax;
                    // anything beyond a slot other than the last one would overwrite an older chunk in the next slot
                    my_bits[s] = constant ? 0u : pack(hs, slot, last_slot ? C.slot_bytes + C.sub : C.slot_bytes);
                    // more than the slot holds: the bits beyond it do not survive the next staging
                    oversize |= my_bits[s] > 8 * C.slot_bytes;
                    ++hs;
                }
            }

            // the ticket of the next batch (see above)
            uint32_t next_ticket = 0;
            if (threadIdx.x == 0) next_ticket = atomicAdd(&C.ctl->ticket, 1u);

            // ---- phase C: subchunk end bits and the chunk's size in the payload area ----
            uint64_t tot16 = 0;
            {
                uint32_t hs = 0;
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    if (!is_huff(s)) continue;
                    uint32_t inc = my_bits[s];
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t x = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                        if (lane >= (uint32_t)o) inc += x;
                    }
                    // A chunk that holds nothing but the fill symbol (the symbol with the all-zero code) takes no bits
                    // at all.  Candidates are the chunks with exactly symbols * length
                    // bits (rare otherwise); their staged symbols are then compared one by one.
                    uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, inc, 31);
                    const uint32_t fill = vol32(&s_fill[tab_slot_idx][hs]);   // fill symbol | its code length << 8
                    if (active && chunk_bits <= C.cs * (fill >> 8)) {  // the last chunk may be shorter
                        const uint32_t syms = (uint32_t)min((uint64_t)C.cs, I.n_syms - (uint64_t)my_c * C.cs);
                        const uint32_t mine = lane * C.sub < syms ? min(C.sub, syms - lane * C.sub) : 0u;
                        if (chunk_bits == syms * (fill >> 8) &&
                            all_symbols_are(smem_u32(stage + hs * C.stage_stride + lane * region) + sym_off, mine, fill & 0xFFu)) {
                            inc = 0;
                            chunk_bits = 0;
                        }
                    }
                    ++hs;
                    cur.end[s] = inc;
                    if (active) {
                        if (C.sub_width == 2) reinterpret_cast<uint16_t*>(I.out + I.lay.sub_end_tab[s] + 64ull * my_c)[lane] = (uint16_t)inc;
                        else reinterpret_cast<uint32_t*>(I.out + I.lay.sub_end_tab[s] + 128ull * my_c)[lane] = inc;
                        tot16 += (chunk_bits + 127) / 128;
                    }
                }
            }
            if (lane == 0) {
                s_tot[it % kRing][warp] = tot16;
                __threadfence_block();
                atomicAdd(&s_cnt[it % kRing], 1u);
            }
            if (threadIdx.x == 0) {
                // another batch of this tensor is handed out right away; anything else is left to the service warp
                const uint32_t r1 = (it + 1) % kRing;
                const bool same = next_ticket < t_end;
                s_ticket[r1] = next_ticket;
                s_tensor[r1] = t;
                s_cbase[r1] = (next_ticket - I.first_batch) * n_workers;
                s_tabslot[r1] = tab_slot_idx;
                __threadfence_block();
                if (same) *reinterpret_cast<volatile uint32_t*>(&s_base_seq) = it + 2;
                *reinterpret_cast<volatile uint32_t*>(&s_ticket_seq) = it + 2;   // after s_base_seq: the service warp reads it first
            }
            if (!n_huff && active) chunk_done(t, 0, 0);             // nothing to copy out: the chunk is complete

            q2 = q1; q1 = q0; q0 = cur;
            ++n_pend;
            slot_idx = last_slot ? 0 : slot_idx + 1;
            if (__any_sync(0xFFFFFFFFu, oversize)) {
                // some subchunk needs more than its slot holds: finish this chunk before anything else is staged.
                // Once everything older has left, a packing that was clipped at the end of its slot is redone from
                // slot 0 with the rest of the region as room.
                while (n_pend > 1 && !failed) failed = !flush_oldest(it + 1);
                if (failed) break;
                if (!last_slot) {
                    uint32_t hs = 0;
#pragma unroll
                    for (int s = 0; s < 2; ++s) {
                        if (!is_huff(s)) continue;
                        pack(hs, 0, 2 * C.sub);
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
        flush_acc();
        if (bad && raise_status(C.ctl, 0, ZC_E_NO_CODE)) C.ctl->failed = item(bad - 1).index + 1;
    }
    __syncthreads();
    if (s_fail && threadIdx.x == 0) raise_status(C.ctl, 0, ZC_E_DEVICE_TIMEOUT);
}

}  // namespace zc

#include "zc_encode_rows.cuh"

using namespace zc;

namespace {

// Chunk size from which on encode_kernel is used instead of the row encoder (which can take chunks up to 8 KiB).
// ZC_ROW_ENCODER_BELOW overrides it (bytes; 0 turns the row encoder off, 8193 gives it everything it can take).
uint32_t row_kernel_limit()
{
    static const uint32_t limit = [] {
        const char* e = getenv("ZC_ROW_ENCODER_BELOW");
        return e ? std::min<uint32_t>((uint32_t)strtoul(e, nullptr, 0), 8193u) : 4096u;
    }();
    return limit;
}

// Launch shape of the row encoder for a plan, or workers == 0 when the plan is not for it (large chunks, no coded
// stream).
RowShape row_shape(const zc_plan_t* p, uint32_t n_huff)
{
    RowShape s{};
    // Measured on one B200 (fractions of the HBM roofline, encode_kernel -> this kernel): 1 KiB chunks 16 -> 22 %,
    // 2 KiB 29 -> 32 %, 4 KiB 49 -> 46 %, 8 KiB 49 -> 41 %: it takes the chunks below 4 KiB.
    if (n_huff == 0 || p->chunk_bytes >= row_kernel_limit()) return s;
    const uint32_t row = p->chunk_bytes / 32;
    s.row_stride = row + 16;
    s.in_bytes = 32 * s.row_stride;
    s.pack1_bytes = n_huff == 2 ? (uint32_t)round_up(32ull * (p->syms_per_sub + p->syms_per_sub / 2 + 4), 16) : 0;
    const uint32_t max_piece = n_huff * (uint32_t)round_up((uint64_t)p->syms_per_chunk * kLmax / 8, 16);
    s.ring_bytes = 4096;
    while (s.ring_bytes < max_piece) s.ring_bytes *= 2;
    // One input buffer per warp: more warps fit, and with about two dozen of them the SM has enough to do while a
    // warp waits for its next chunk.  (Two buffers, the next chunk travelling while this one is packed, leave room
    // for 16 warps at 4 KiB chunks, which measured slower.)
    s.n_buf = 1;
    const size_t per_warp = s.n_buf * (size_t)s.in_bytes + s.pack1_bytes + s.ring_bytes;
    const size_t fixed = (size_t)4 * kTabSlots * 256 * n_huff + 12288 /* static shared and reserve */;
    s.workers = (uint32_t)std::min<size_t>(kRowMaxWorkers, (kMaxSmem - fixed) / per_warp);
    if (s.workers < 4) { s.workers = 0; return s; }
    s.smem = (size_t)4 * kTabSlots * 256 * n_huff + s.workers * per_warp;
    return s;
}

#if ZC_DEBUG_CHECKS
// development build: the address ranges the launch may touch (hulls over the tensors of the launch)
template <int N_ITEMS>
void dbg_ranges_of(const EncParamsT<N_ITEMS>& P, cudaStream_t st)
{
    DbgHull rd, wr, ws;
    const uint32_t n = N_ITEMS > 1 ? P.c.n_tensors : 1;
    for (uint32_t i = 0; i < n; ++i) {
        const EncItem& it = P.item[i];
        rd.add(it.in, it.input_bytes);
        rd.add(it.base, it.input_bytes);
        // no container is larger than its tables plus 12 bits per symbol of either stream, padding and guard
        wr.add(it.out, it.lay.payload_off + 3 * it.n_syms + 32ull * it.n_chunks + 64);
        if (P.c.counters) ws.add(P.c.counters + it.index, sizeof(TensorCounters));
        if (N_ITEMS > 1 && P.c.tables) ws.add(P.c.tables + it.table, sizeof(EncTables));
    }
    ws.add(P.c.ctl, sizeof(Control));
    ws.add(P.c.flags, 8ull * std::max<uint32_t>(P.c.total_batches, 1));
    dbg_set_ranges(st, rd.ptr(), rd.bytes(), wr.ptr(), wr.bytes(), ws.ptr(), ws.bytes());
}
#endif

template <int N_ITEMS>
cudaError_t launch_encode_rows(const EncParamsT<N_ITEMS>& P, uint32_t format, const RowShape& sh, const zc_plan_t* p0, cudaStream_t st)
{
    RowParams RP{sh.row_stride, sh.in_bytes, sh.pack1_bytes, sh.ring_bytes, p0->chunk_bytes / 512, sh.n_buf};
    const uint32_t want = std::max<uint32_t>(P.c.total_batches, 1);
    const uint32_t grid = std::min<uint32_t>(want, (uint32_t)sm_count());
    cudaError_t e = cudaSuccess;
    auto launch = [&](auto kern) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh.smem);
        if (e != cudaSuccess) return;
#if ZC_DEBUG_CHECKS
        dbg_ranges_of(P, st);
#endif
        kern<<<grid, (sh.workers + 2) * 32, sh.smem, st>>>(P, RP);
        e = cudaGetLastError();
    };
    const bool h0 = P.c.mode[0] == ZC_MODE_HUFF, h1 = P.c.mode[1] == ZC_MODE_HUFF;
#define ZC_ENC_CASE(F)                                                                  \
    if (h0 && h1) launch(encode_rows_kernel<F, N_ITEMS, true, true>);                  \
    else if (h0) launch(encode_rows_kernel<F, N_ITEMS, true, false>);                  \
    else launch(encode_rows_kernel<F, N_ITEMS, false, true>);
    switch (format) {
    case ZC_FMT_BF16: ZC_ENC_CASE(ZC_FMT_BF16) break;
    case ZC_FMT_FP8_E4M3: case ZC_FMT_FP8_E5M2: ZC_ENC_CASE(ZC_FMT_FP8_E4M3) break;
    case ZC_FMT_SCALE_U8: ZC_ENC_CASE(ZC_FMT_SCALE_U8) break;
    default: ZC_ENC_CASE(ZC_FMT_FP4_E2M1) break;
    }
#undef ZC_ENC_CASE
    return e;
}

// Shared-memory shape of a launch for given chunk geometry, number of coded streams and slot size.
constexpr uint32_t kSlotsNarrow = 0, kSlotsWide = 1, kSlotsHalf = 2;    // pack slots of 8 / 12 / 4 bits per symbol
struct EncShape { uint32_t n_slots, slot_bytes, region_bytes, stage_stride, workers, per_sm; size_t smem; };

// slots: kSlotsNarrow / kSlotsWide / kSlotsHalf (see slot_class)
zc_status enc_shape(const zc_plan_t* p, uint32_t n_huff, uint32_t slots, EncShape* out)
{
    EncShape s{};
    const size_t fixed = (size_t)4 * kTabSlots * 256 * std::max<uint32_t>(n_huff, 1);
    s.slot_bytes = slots == kSlotsWide ? p->syms_per_sub + p->syms_per_sub / 2 : p->syms_per_sub;
    // pack slots per lane region: first as many resident blocks of 8 worker warps per SM as possible (up to 3),
    // then as many slots (up to 3) as that number of blocks leaves room for
    s.n_slots = 1;
    uint32_t best_score = 0;
    for (uint32_t ns = 1; ns <= 3; ++ns) {
        const size_t block = fixed + (size_t)kEncMaxWorkers * std::max<uint32_t>(n_huff, 1) * kSubs * (ns * s.slot_bytes + p->syms_per_sub + 4);
        const uint32_t blocks = (uint32_t)std::min<size_t>((kMaxSmem + 1024) / (block + 2048 + 1024), 3);
        // a second slot is worth a resident block (with one slot every turn waits for its look-back), a third is not
        const uint32_t score = blocks * std::min<uint32_t>(ns, 2) * 4 + ns;
        if (blocks > 0 && score >= best_score) { best_score = score; s.n_slots = ns; }
    }
    // Long subchunks: lane regions of (slots + 1) * sub bytes leave room for a handful of warps per SM.  One slot of
    // half a subchunk is enough to be correct (a lane writes at most 1.5 bytes per symbol it has read, so packing from
    // the start of a region of 1.5 * sub bytes never overtakes the symbols still to be read); a chunk whose bits do
    // not fit the slot leaves at once instead of waiting up to three turns.  Chosen (slot_class) for code tables that
    // promise well under 4 bits per symbol: where most chunks overflow the slot every turn waits for its own look-back.
    if (slots == kSlotsHalf) {
        s.n_slots = 1;
        s.slot_bytes = p->syms_per_sub / 2;
    }
    s.region_bytes = s.n_slots * s.slot_bytes + p->syms_per_sub + 4;
    s.stage_stride = kSubs * s.region_bytes;
    const size_t per_warp = std::max<size_t>((size_t)n_huff * s.stage_stride, 16);
    // blocks of up to 8 worker warps (a batch of 8 consecutive chunks) plus the service warp; several
    // blocks per SM so that loading, packing and copy-out phases of different blocks overlap
    s.workers = (uint32_t)std::min<size_t>(kEncMaxWorkers, (kMaxSmem - fixed - 2048) / per_warp);
    if (s.workers == 0) return ZC_E_UNSUPPORTED;
    s.smem = fixed + s.workers * per_warp;
    s.per_sm = std::max<uint32_t>((uint32_t)std::min<size_t>((kMaxSmem + 1024) / (s.smem + 2048 + 1024), 3), 1u);
    *out = s;
    return ZC_OK;
}

// Wide pack slots (12 bits per symbol) for code tables whose codes are long on average (decided per stream when
// the codebook is built).  Shorter codes get slots of 8 bits per symbol and the slow path for the rare subchunk
// that needs more; very short codes in long subchunks get one slot of 4 bits per symbol (enc_shape says why).
uint32_t slot_class(const zc_plan_t* p, const zc_codebook_t* cb, const uint32_t mode[2])
{
    const bool h0 = mode[0] == ZC_MODE_HUFF, h1 = mode[1] == ZC_MODE_HUFF;
    if ((h0 && cb->wide[0]) || (h1 && cb->wide[1])) return kSlotsWide;
    // subchunks of 256 symbols and more (chunks from 16 KiB): half-size slots leave room for twice the warps
    if ((h0 || h1) && p->syms_per_sub >= 256 && (!h0 || cb->brief[0]) && (!h1 || cb->brief[1])) return kSlotsHalf;
    return kSlotsNarrow;
}

void fill_common(EncCommon& c, const zc_plan_t* p, const uint32_t mode[2], const EncShape& sh)
{
    c.cs = p->syms_per_chunk; c.sub = p->syms_per_sub; c.chunk_bytes = p->chunk_bytes;
    c.format = p->format; c.group = p->group;
    c.mode[0] = mode[0]; c.mode[1] = mode[1];
    c.n_slots = sh.n_slots; c.slot_bytes = sh.slot_bytes; c.region_bytes = sh.region_bytes; c.stage_stride = sh.stage_stride;
    c.sub_width = sub_end_width(p->chunk_bytes);
    c.spin_limit = test_knobs().spin_limit;
    c.sub_magic = (uint32_t)(((1ull << 32) + p->syms_per_sub - 1) / p->syms_per_sub);
    c.stage_step = 256 % p->syms_per_sub == 0 ? (256 / p->syms_per_sub) * sh.region_bytes : 0;
}

void fill_item(EncItem& it, const zc_plan_t* p, const uint32_t mode[2], const void* d_in, const void* d_base, void* d_out,
               uint32_t first_batch, uint32_t index, uint32_t table)
{
    it.in = (const uint8_t*)d_in;
    it.base = (const uint8_t*)d_base;
    it.out = (uint8_t*)d_out;
    it.input_bytes = p->input_bytes; it.n_syms = p->n_syms; it.n_elems = p->n_elems;
    it.n_chunks = p->n_chunks;
    it.first_batch = first_batch;
    it.index = index;
    it.table = table;
    it.lay = make_layout(*p, mode);
}

void fill_tables(EncTables& T, const zc_codebook_t* cb)
{
    static_assert(sizeof(T.enc) == sizeof(cb->enc), "table layout");
    std::memcpy(T.enc, cb->enc, sizeof(T.enc));
}

template <int N_ITEMS>
cudaError_t launch_encode(const EncParamsT<N_ITEMS>& P, uint32_t format, const EncShape& sh, cudaStream_t st)
{
    const uint32_t want = std::max<uint32_t>(P.c.total_batches, 1);
    const uint32_t grid = std::min<uint32_t>(want, (uint32_t)sm_count() * sh.per_sm);
    cudaError_t e = cudaSuccess;
    auto launch = [&](auto kern) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh.smem);
        if (e != cudaSuccess) return;
#if ZC_DEBUG_CHECKS
        dbg_ranges_of(P, st);
#endif
        kern<<<grid, (sh.workers + 1) * 32, sh.smem, st>>>(P);
        e = cudaGetLastError();
    };
    const bool h0 = P.c.mode[0] == ZC_MODE_HUFF, h1 = P.c.mode[1] == ZC_MODE_HUFF;
#define ZC_ENC_CASE(F)                                                                  \
    if (h0 && h1) launch(encode_kernel<F, N_ITEMS, true, true>);                       \
    else if (h0) launch(encode_kernel<F, N_ITEMS, true, false>);                       \
    else if (h1) launch(encode_kernel<F, N_ITEMS, false, true>);                       \
    else launch(encode_kernel<F, N_ITEMS, false, false>);
    switch (format) {
    case ZC_FMT_BF16: ZC_ENC_CASE(ZC_FMT_BF16) break;
    case ZC_FMT_FP8_E4M3: case ZC_FMT_FP8_E5M2: ZC_ENC_CASE(ZC_FMT_FP8_E4M3) break;
    case ZC_FMT_SCALE_U8: ZC_ENC_CASE(ZC_FMT_SCALE_U8) break;
    default: ZC_ENC_CASE(ZC_FMT_FP4_E2M1) break;
    }
#undef ZC_ENC_CASE
    return e;
}

// Workspace of a batched call: control block | counters[n] | look-back words[batches] | tables[n].  Everything
// before the tables starts from zero (one clear), the tables are uploaded.
struct BatchLayout { size_t counters, flags, tables, total; };

BatchLayout batch_layout(uint32_t n_tensors, uint64_t total_batches)
{
    BatchLayout L{};
    L.counters = kControlBytes;
    L.flags = (size_t)round_up(L.counters + sizeof(TensorCounters) * (uint64_t)n_tensors, 256);
    L.tables = (size_t)round_up(L.flags + 8ull * total_batches, 256);
    L.total = (size_t)round_up(L.tables + sizeof(EncTables) * (uint64_t)n_tensors, 256);
    return L;
}

// Host-to-device copy of the code tables of a batched call.  A large copy from pageable memory holds the host
// until the stream has drained, which would make an asynchronous call wait for the previous call's kernel; so
// the tables go through a pinned staging buffer, one per calling thread, that is reused once the previous copy
// out of it has been done (an event says so).  The buffer is never freed (a thread's last CUDA calls may come
// after the runtime has shut down).  Without pinned memory the copy falls back to the pageable one.
struct TableStage { void* ptr = nullptr; size_t cap = 0; cudaEvent_t done = nullptr; int device = -1; };

cudaError_t upload_tables(void* d_dst, const void* h_src, size_t bytes, cudaStream_t st)
{
    static thread_local TableStage stage;
    if (bytes <= 48 * 1024)                      // small copies leave the caller's memory at once anyway
        return cudaMemcpyAsync(d_dst, h_src, bytes, cudaMemcpyHostToDevice, st);
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return cudaErrorUnknown;
    if (stage.done) {
        if (cudaEventSynchronize(stage.done) != cudaSuccess) return cudaErrorUnknown;
        if (stage.device != device) { cudaEventDestroy(stage.done); stage.done = nullptr; }
    }
    if (stage.cap < bytes) {
        if (stage.ptr) cudaFreeHost(stage.ptr);
        stage.ptr = nullptr;
        stage.cap = 0;
        const size_t want = (size_t)round_up(bytes, 1u << 18);
        if (cudaHostAlloc(&stage.ptr, want, cudaHostAllocPortable) == cudaSuccess) stage.cap = want;
        else { stage.ptr = nullptr; (void)cudaGetLastError(); }
    }
    if (!stage.ptr) return cudaMemcpyAsync(d_dst, h_src, bytes, cudaMemcpyHostToDevice, st);
    if (!stage.done) {
        if (cudaEventCreateWithFlags(&stage.done, cudaEventDisableTiming) != cudaSuccess) {
            stage.done = nullptr;
            (void)cudaGetLastError();
            return cudaMemcpyAsync(d_dst, h_src, bytes, cudaMemcpyHostToDevice, st);
        }
        stage.device = device;
    }
    std::memcpy(stage.ptr, h_src, bytes);
    const cudaError_t e = cudaMemcpyAsync(d_dst, stage.ptr, bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return e;
    return cudaEventRecord(stage.done, st);
}

// Upper bound of the batches a tensor is cut into, whatever the modes of its streams turn out to be.
uint64_t max_batches_of(const zc_plan_t* p)
{
    EncShape sh;
    if (enc_shape(p, 2, kSlotsWide, &sh) != ZC_OK) return p->n_chunks;
    uint64_t workers = sh.workers;
    for (uint32_t n_huff = 1; n_huff <= 2; ++n_huff) {
        const RowShape rs = row_shape(p, n_huff);
        if (rs.workers) workers = std::min<uint64_t>(workers, rs.workers);
    }
    return (p->n_chunks + workers - 1) / workers;
}

}  // namespace

namespace zc {
void debug_counts_encode(uint32_t out[2])
{
#if ZC_DEBUG_CHECKS
    dbg_read_counts(out);
#else
    (void)out;
#endif
}
}  // namespace zc

extern "C" {

uint32_t zc_test_encoder_workers(const zc_plan_t* p, uint32_t n_coded, uint32_t wide_slots)
{
    EncShape sh;
    if (!p || n_coded > 2 || wide_slots > kSlotsHalf || enc_shape(p, n_coded, wide_slots, &sh) != ZC_OK) return 0;
    return sh.workers;
}

zc_status zc_compress(const zc_plan_t* p, const zc_codebook_t* cb, const void* d_in, void* d_out, size_t out_capacity,
                      void* d_workspace, uint64_t* h_out_bytes, void* cuda_stream)
{
    return zc_compress_xor(p, cb, d_in, nullptr, d_out, out_capacity, d_workspace, h_out_bytes, cuda_stream);
}

zc_status zc_compress_xor(const zc_plan_t* p, const zc_codebook_t* cb, const void* d_in, const void* d_base, void* d_out,
                          size_t out_capacity, void* d_workspace, uint64_t* h_out_bytes, void* cuda_stream)
{
    if (!p || !cb || !d_out || !d_workspace || (!d_in && p->n_elems)) return ZC_E_INVALID_ARG;
    if (!aligned16(d_in) || !aligned16(d_base) || !aligned16(d_out) || !aligned16(d_workspace)) return ZC_E_INVALID_ARG;
    if (out_capacity < zc_max_compressed_bytes(p)) return ZC_E_BUFFER_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    uint32_t mode[2], n_huff = 0;
    for (int s = 0; s < 2; ++s) {
        // an empty tensor has no symbols to code: both streams are stored raw
        mode[s] = p->n_syms ? cb->mode[s] : (uint32_t)ZC_MODE_RAW;
        n_huff += mode[s] == ZC_MODE_HUFF;
    }
    EncShape sh;
    const zc_status ss = enc_shape(p, n_huff, slot_class(p, cb, mode), &sh);
    if (ss != ZC_OK) return ss;
    const RowShape rows = d_base ? RowShape{} : row_shape(p, n_huff);
    if (rows.workers) sh.workers = rows.workers;                 // chunks per batch

    static thread_local EncParamsT<1> P;
    P.c = EncCommon{};
    fill_common(P.c, p, mode, sh);
    P.c.ctl = (Control*)d_workspace;
    P.c.counters = &P.c.ctl->tc;
    P.c.flags = (unsigned long long*)((uint8_t*)d_workspace + kControlBytes);
    P.c.tables = nullptr;
    P.c.n_tensors = 1;
    P.c.total_batches = (uint32_t)((p->n_chunks + (uint64_t)sh.workers - 1) / sh.workers);
    fill_item(P.item[0], p, mode, d_in, d_base, d_out, 0, 0, 0);
    fill_tables(P.table, cb);

    if (cudaMemsetAsync(d_workspace, 0, kControlBytes + 8ull * P.c.total_batches, st) != cudaSuccess) return ZC_E_CUDA;
    if (test_knobs().first_ticket) {             // test hook: the tickets start late, batch 0 is never packed
        static uint32_t first;
        first = test_knobs().first_ticket;
        if (cudaMemcpyAsync(&((Control*)d_workspace)->ticket, &first, sizeof(first), cudaMemcpyHostToDevice, st) != cudaSuccess) return ZC_E_CUDA;
    }
    if ((rows.workers ? launch_encode_rows<1>(P, p->format, rows, p, st) : launch_encode<1>(P, p->format, sh, st)) != cudaSuccess) return ZC_E_CUDA;

    if (h_out_bytes) {
        Control h;
        if (cudaMemcpyAsync(&h, d_workspace, sizeof(Control), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZC_E_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return ZC_E_CUDA;
        if (h.status & 0xFF) return (zc_status)(h.status & 0xFF);
        *h_out_bytes = h.tc.total16;
    }
    return ZC_OK;
}

size_t zc_compress_batch_workspace_bytes(uint32_t n_tensors, const zc_plan_t* const* plans)
{
    if (!plans) return 0;
    uint64_t batches = 0;
    for (uint32_t t = 0; t < n_tensors; ++t) {
        if (!plans[t]) return 0;
        batches += max_batches_of(plans[t]);
    }
    return batch_layout(n_tensors, batches).total;
}

zc_status zc_compress_batch(uint32_t n_tensors, const zc_plan_t* const* plans, const zc_codebook_t* const* codebooks,
                            const void* const* d_in, void* const* d_out, const size_t* out_capacity,
                            void* d_workspace, size_t workspace_bytes, uint64_t* h_out_bytes, void* cuda_stream)
{
    return zc_compress_batch_xor(n_tensors, plans, codebooks, d_in, nullptr, d_out, out_capacity, d_workspace, workspace_bytes,
                                 h_out_bytes, cuda_stream);
}

zc_status zc_compress_batch_xor(uint32_t n_tensors, const zc_plan_t* const* plans, const zc_codebook_t* const* codebooks,
                                const void* const* d_in, const void* const* d_base, void* const* d_out,
                                const size_t* out_capacity, void* d_workspace, size_t workspace_bytes,
                                uint64_t* h_out_bytes, void* cuda_stream)
{
    if (!d_workspace || !aligned16(d_workspace)) return ZC_E_INVALID_ARG;
    if (n_tensors == 0) return ZC_OK;
    if (!plans || !codebooks || !d_in || !d_out || !out_capacity) return ZC_E_INVALID_ARG;
    uint64_t max_batches = 0;
    for (uint32_t t = 0; t < n_tensors; ++t) {
        const zc_plan_t* p = plans[t];
        if (!p || !codebooks[t] || !d_out[t] || (!d_in[t] && p->n_elems)) return ZC_E_INVALID_ARG;
        if (!aligned16(d_in[t]) || !aligned16(d_out[t]) || (d_base && !aligned16(d_base[t]))) return ZC_E_INVALID_ARG;
        if (p->format != plans[0]->format || p->chunk_bytes != plans[0]->chunk_bytes) return ZC_E_INVALID_ARG;
        if (out_capacity[t] < zc_max_compressed_bytes(p)) return ZC_E_BUFFER_TOO_SMALL;
        max_batches += max_batches_of(p);
    }
    const BatchLayout L = batch_layout(n_tensors, max_batches);
    if (workspace_bytes < L.total) return ZC_E_BUFFER_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint8_t* ws = (uint8_t*)d_workspace;
    const zc_plan_t* p0 = plans[0];

    // control block, counters and look-back words start from zero
    if (cudaMemsetAsync(ws, 0, L.tables, st) != cudaSuccess) return ZC_E_CUDA;
    // the code tables are uploaded in one copy, one per distinct codebook (the K/V pages of a step share theirs)
    static thread_local std::vector<EncTables> h_tables;
    static thread_local std::vector<uint32_t> table_of;          // per tensor: its tables among the uploaded ones
    static thread_local std::vector<uint8_t> table_slots;        // per uploaded table: the slot class its codes ask for
    static thread_local std::unordered_map<const zc_codebook_t*, uint32_t> seen;
    h_tables.clear(); table_slots.clear(); seen.clear();
    table_of.resize(n_tensors);
    for (uint32_t t = 0; t < n_tensors; ++t) {
        auto found = seen.find(codebooks[t]);
        if (found == seen.end()) {
            found = seen.emplace(codebooks[t], (uint32_t)h_tables.size()).first;
            h_tables.emplace_back();
            fill_tables(h_tables.back(), codebooks[t]);
            const uint32_t m[2] = {codebooks[t]->mode[0], codebooks[t]->mode[1]};
            table_slots.push_back((uint8_t)slot_class(p0, codebooks[t], m));
        }
        table_of[t] = found->second;
    }
    if (upload_tables(ws + L.tables, h_tables.data(), sizeof(EncTables) * h_tables.size(), st) != cudaSuccess) return ZC_E_CUDA;

    // one launch per combination of stream modes and slot size (the kernel's shared-memory layout depends on
    // them) and per kEncBatchMax tensors of it
    static thread_local EncParamsT<(int)kEncBatchMax> P;
    uint64_t flag_base = 0;
    bool first_launch = true;
    static thread_local std::vector<uint8_t> group;              // per tensor: mode0 | mode1 << 1 | slot class << 2
    group.resize(n_tensors);
    for (uint32_t t = 0; t < n_tensors; ++t) {
        const bool any = plans[t]->n_syms != 0;                  // an empty tensor: both streams raw
        const uint32_t m[2] = {any ? codebooks[t]->mode[0] : (uint32_t)ZC_MODE_RAW, any ? codebooks[t]->mode[1] : (uint32_t)ZC_MODE_RAW};
        const uint32_t slots = (m[0] == ZC_MODE_HUFF || m[1] == ZC_MODE_HUFF) ? table_slots[table_of[t]] : kSlotsNarrow;
        group[t] = (uint8_t)(m[0] | (m[1] << 1) | (slots << 2));
    }
    // the launch shapes of the combinations that occur, checked before anything is launched
    bool combo_used[12] = {};
    for (uint32_t t = 0; t < n_tensors; ++t) combo_used[group[t]] = true;
    for (uint32_t combo = 0; combo < 12; ++combo) {
        EncShape sh;
        if (combo_used[combo] && enc_shape(p0, (combo & 1u) + ((combo >> 1) & 1u), combo >> 2, &sh) != ZC_OK) return ZC_E_UNSUPPORTED;
    }
    for (uint32_t combo = 0; combo < 12; ++combo) {
        if (!combo_used[combo]) continue;
        const uint32_t mode[2] = {combo & 1u, (combo >> 1) & 1u};
        const uint32_t n_huff = (mode[0] == ZC_MODE_HUFF) + (mode[1] == ZC_MODE_HUFF);
        auto in_combo = [&](uint32_t t) { return group[t] == combo; };
        EncShape sh;
        const zc_status ss = enc_shape(p0, n_huff, combo >> 2, &sh);
        if (ss != ZC_OK) return ss;
        bool any_base = false;
        if (d_base) for (uint32_t i = 0; i < n_tensors; ++i) any_base = any_base || d_base[i] != nullptr;
        const RowShape rows = any_base ? RowShape{} : row_shape(p0, n_huff);
        if (rows.workers) sh.workers = rows.workers;
        uint32_t t = 0;
        while (t < n_tensors) {
            P.c = EncCommon{};
            fill_common(P.c, p0, mode, sh);
            uint32_t n = 0;
            uint64_t batches = 0;
            for (; t < n_tensors && n < kEncBatchMax; ++t) {
                if (!in_combo(t)) continue;
                const uint64_t nb = (plans[t]->n_chunks + (uint64_t)sh.workers - 1) / sh.workers;
                if (batches + nb >= (1ull << 32)) break;
                fill_item(P.item[n], plans[t], mode, d_in[t], d_base ? d_base[t] : nullptr, d_out[t], (uint32_t)batches, t, table_of[t]);
                batches += nb;
                ++n;
            }
            if (n == 0) {
                if (t < n_tensors) return ZC_E_UNSUPPORTED;      // a single tensor with 2^32 batches or more
                break;
            }
            P.c.ctl = (Control*)ws;
            P.c.counters = (TensorCounters*)(ws + L.counters);
            P.c.tables = (const EncTables*)(ws + L.tables);
            P.c.flags = (unsigned long long*)(ws + L.flags) + flag_base;
            P.c.n_tensors = n;
            P.c.total_batches = (uint32_t)batches;
            flag_base += batches;
            // the ticket counter restarts for every launch (the first one finds it cleared)
            if (!first_launch && cudaMemsetAsync(&((Control*)ws)->ticket, 0, sizeof(uint32_t), st) != cudaSuccess) return ZC_E_CUDA;
            first_launch = false;
            if ((rows.workers ? launch_encode_rows<(int)kEncBatchMax>(P, p0->format, rows, p0, st)
                              : launch_encode<(int)kEncBatchMax>(P, p0->format, sh, st)) != cudaSuccess) return ZC_E_CUDA;
        }
    }

    if (h_out_bytes) {
        // control block and counters lie next to each other: one copy
        static thread_local std::vector<uint8_t> h_state;
        const size_t bytes = L.counters + sizeof(TensorCounters) * (size_t)n_tensors;
        h_state.resize(bytes);
        if (cudaMemcpyAsync(h_state.data(), ws, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZC_E_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return ZC_E_CUDA;
        Control h;
        std::memcpy(&h, h_state.data(), sizeof(Control));
        if (h.status & 0xFF) return (zc_status)(h.status & 0xFF);
        for (uint32_t t = 0; t < n_tensors; ++t) {
            TensorCounters tc;
            std::memcpy(&tc, h_state.data() + L.counters + sizeof(TensorCounters) * (size_t)t, sizeof(tc));
            h_out_bytes[t] = tc.total16;
        }
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
std::atomic<void*> g_noalloc_ptr[kMaxDevices];

// Device address of the scratch array on the current device; looked up once per device (two host threads that
// make the first call together both look it up and store the same address).
zc_status noalloc_scratch(void** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ZC_E_CUDA;
    void* ptr = g_noalloc_ptr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return ZC_E_CUDA;
        g_noalloc_ptr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
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

zc_status zc_noalloc_status(void* cuda_stream)
{
    void* scratch = nullptr;
    const zc_status st = noalloc_scratch(&scratch);
    if (st != ZC_OK) return st;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    unsigned long long word[2] = {0, 0};            // status, call id
    if (cudaMemcpyAsync(word, scratch, sizeof(word), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return ZC_E_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return ZC_E_CUDA;
    return (word[0] >> 8) == word[1] ? (zc_status)(word[0] & 0xFF) : ZC_OK;
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
