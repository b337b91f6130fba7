// Row encoder: the encoder kernel for chunks of up to 8 KiB without a base tensor (included by zc_encode.cu).
//
// Same container, same batches and look-back words as encode_kernel; what differs is how the data moves:
//   in    every worker warp brings its next chunk into shared memory with 16-byte asynchronous copies
//         (cp.async, coalesced in global memory) one turn ahead, laid out as one row per lane = the lane's
//         subchunk (chunk_bytes / 32 input bytes, rows padded by 16 bytes so that 16-byte row reads of the
//         32 lanes do not collide)
//   pack  a lane reads its row 16 bytes at a time, splits the fields in registers, stores the raw stream's
//         bytes straight to the container and packs the coded stream's bits over the part of the row it has
//         already read (at most 12 of every 16 bytes read are written)
//   out   after the warp scan of the bit counts every lane shifts its bits into place inside a compact piece
//         in a ring in shared memory; the service warp, which knows the chunk's position once the batch's
//         look-back is done, sends the piece to the container with one bulk copy (cp.async.bulk shared ->
//         global, non-multicast)
// So no symbols are staged, a packed chunk waits for its position as a few hundred bytes instead of a slot per
// lane, workers never wait for a look-back (only for ring space, which the service warp frees as soon as a bulk
// copy has read its piece), and the service warp takes the tickets of the block's batches two ahead, which is
// what lets a warp request its next input a whole turn early.  One block of up to 16 worker warps per SM.
#pragma once

namespace zc {

constexpr uint32_t kRowMaxWorkers = 22;      // worker warps per block; one block per SM (24 warps of at most 85 registers)
constexpr uint32_t kRowRing = 16;            // batches of a block whose bookkeeping is alive at the same time: a batch's slot is
                                             // reused 16 batches later, when every worker has long sent its piece off (at most five
                                             // batches wait for their place, and a worker sends what has been placed at every turn)
constexpr uint32_t kRowSleep = 400;          // nanoseconds a waiting warp sleeps between two looks: polling costs issue slots the
                                             // packing warps need
constexpr uint32_t kRowAhead = 2;            // batches dealt out beyond the newest one a worker has begun
constexpr int kRowLook = 5;                  // look-back rounds cover 32 * kRowLook predecessors: more than the resident blocks

struct RowShape {
    uint32_t workers;        // worker warps per block (= chunks per batch)
    uint32_t row_stride;     // bytes from one lane's row to the next: chunk_bytes / 32 + 16
    uint32_t in_bytes;       // one input buffer of a warp: 32 rows
    uint32_t pack1_bytes;    // both streams coded: the second stream's pack rows of a warp (0 otherwise)
    uint32_t ring_bytes;     // the warp's piece ring (power of two)
    uint32_t n_buf;          // input buffers per warp (1 or 2)
    size_t smem;
};

struct RowParams {           // appended to the common parameters
    uint32_t row_stride, in_bytes, pack1_bytes, ring_bytes, units;   // units = 16-byte units per row
    uint32_t n_buf;          // input buffers per warp: 2 = the next chunk travels while this one is packed, 1 = while it waits
};

__device__ __forceinline__ void cp_async16(uint32_t dst_s, const void* src, uint32_t src_bytes)
{
    ZC_DBG_SHARED(dst_s, 16, return); if (src_bytes) ZC_DBG_GLOBAL(src, src_bytes, 16, false, return);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst_s), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_s2g(void* dst, uint32_t src_s, uint32_t bytes)
{
    ZC_DBG_GLOBAL(dst, bytes, 16, true, return); ZC_DBG_SHARED(src_s, 16, return); ZC_DBG_SHARED(src_s + bytes - 16, 16, return);
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" :: "l"(dst), "r"(src_s), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint4 lds128e(uint32_t addr)
{
    ZC_DBG_SHARED(addr, 16, return make_uint4(0, 0, 0, 0));
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// Append `len` bits (left-aligned in `code`, zero below them) to a lane's accumulator; a completed word goes to
// shared address waddr.  hi holds the nb (< 32) pending bits left-aligned.
__device__ __forceinline__ void put_bits_row(uint32_t code, uint32_t len, uint32_t& hi, uint32_t& nb, uint32_t& waddr)
{
    hi |= code >> nb;
    const uint32_t lo = __funnelshift_r(0, code, nb);           // the bits that do not fit: code << (32 - nb), 0 if nb == 0
    const uint32_t n = nb + len;
    const bool full = n >= 32;
    sts32_if(full, waddr, hi);
    waddr += full ? 4 : 0;
    hi = full ? lo : hi;
    nb = n & 31;
}

template <int FMT, int N_ITEMS, bool H0, bool H1>
__global__ void __launch_bounds__((kRowMaxWorkers + 2) * 32, 1)
encode_rows_kernel(const __grid_constant__ EncParamsT<N_ITEMS> P, const __grid_constant__ RowParams RP)
{
    extern __shared__ __align__(16) uint8_t smem[];
    const EncCommon& C = P.c;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n_workers = (blockDim.x >> 5) - 2;            // then the dealer warp and the placer warp
    const bool service = warp >= n_workers;
    constexpr uint32_t n_huff = (H0 ? 1u : 0u) + (H1 ? 1u : 0u);
    static_assert(n_huff >= 1, "tensors without a coded stream go through encode_kernel");
    auto is_huff = [](const int s) constexpr { return s == 0 ? H0 : H1; };

    // shared: tables[kTabSlots][n_huff][256] | per worker warp: in[2][in_bytes] | pack1 | ring
    uint32_t* tabs = reinterpret_cast<uint32_t*>(smem);
    constexpr uint32_t tab_words = 256 * n_huff;
    const uint32_t per_warp = RP.n_buf * RP.in_bytes + RP.pack1_bytes + RP.ring_bytes;
    uint8_t* const warp_base = smem + 4 * kTabSlots * tab_words + (size_t)(service ? 0 : warp) * per_warp;
    const uint32_t ring_words = RP.ring_bytes / 4;

    __shared__ uint32_t s_tensor[kRowRing], s_cbase[kRowRing], s_tabslot[kRowRing], s_cnt[kRowRing], s_ticket[kRowRing];
    __shared__ uint32_t s_base_seq, s_fail;
    __shared__ uint32_t s_fill[kTabSlots][2];
    __shared__ uint32_t s_tot[kRowRing][kRowMaxWorkers];        // size of worker w's chunk in 16-byte units (both streams)
    __shared__ uint32_t s_p0[kRowRing][kRowMaxWorkers];         // of which stream 0's piece
    __shared__ uint32_t s_roff[kRowRing][kRowMaxWorkers];       // where the chunk's pieces start in the worker's ring (16-byte units)
    __shared__ uint16_t s_bits[kRowRing][kRowMaxWorkers][2];    // payload bits of the chunk per stream (below 65536 for chunks up to 8 KiB)
    __shared__ unsigned long long s_off[kRowRing][kRowMaxWorkers];   // where worker w's chunk goes in the payload area (16-byte units)
    __shared__ uint32_t s_off_seq;                              // batches of this block that have been placed
    __shared__ uint32_t s_agg_seq;                              // batches of this block whose size has been published
    __shared__ uint32_t s_lead;                                 // batches of this block that some worker has begun

    if (threadIdx.x < kRowRing) s_cnt[threadIdx.x] = 0;
    if (threadIdx.x == 0) { s_fail = 0; s_base_seq = 0; s_off_seq = 0; s_agg_seq = 0; s_lead = 0; }
    __syncthreads();

    auto vol32 = [](const uint32_t* p) { return *reinterpret_cast<const volatile uint32_t*>(p); };
    // the same value in every lane (decisions that lead to warp-wide operations must not differ between lanes)
    auto uni32 = [](const uint32_t* p) { return __shfl_sync(0xFFFFFFFFu, *reinterpret_cast<const volatile uint32_t*>(p), 0); };
    auto item = [&](const uint32_t t) -> const EncItem& { return P.item[N_ITEMS == 1 ? 0u : t]; };
    auto counters = [&](const uint32_t t) -> TensorCounters* { return C.counters + (N_ITEMS == 1 ? 0u : P.item[t].index); };

    if (warp == n_workers) {
        // =========================== the dealer warp ===========================
        // Takes the block's tickets, turns them into batches for the workers (tensor, first chunk, code table) and
        // publishes a batch's size the moment all its workers have posted theirs.  Nothing here waits for global
        // memory except the ticket itself, which is requested one loop turn before it is used.
        if (blockIdx.x == 0 && lane == 0)
            for (uint32_t t = 0; t < C.n_tensors; ++t)
                if (item(t).n_chunks == 0) write_header(C, item(t), counters(t));

        uint32_t handed = 0, agg_posted = 0;
        uint32_t tcur = 0, idle = 0;
        uint32_t tab_tensor = kNoTensor, tab_slot = 0;
        uint32_t slot_last0 = 0, slot_last1 = 0, slot_last2 = 0, slot_last3 = 0;   // 1 + last batch that used slot k
        bool ended = false;
        uint32_t ticket = 0;
        int ticket_state = 0;                                     // 0 none, 1 requested, 2 here
        auto load_next_slot = [&](const uint32_t t, const uint32_t packed_now) -> bool {
            const uint32_t nslot = (tab_slot + 1) % kTabSlots;
            const uint32_t last = nslot == 0 ? slot_last0 : nslot == 1 ? slot_last1 : nslot == 2 ? slot_last2 : slot_last3;
            if (packed_now < last) return false;                 // a worker may still pack with the table that is there
            uint32_t* tab = tabs + nslot * tab_words;
            uint32_t hs = 0;
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                if (!is_huff(s)) continue;
                const uint32_t* src;
                if constexpr (N_ITEMS == 1) src = P.table.enc[s]; else src = C.tables[item(t).table].enc[s];
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
                    if (lane == 0) s_fill[nslot][hs] = who ? fill : 0xFF00u;
                }
                ++hs;
            }
            __syncwarp();
            return true;
        };
        for (;;) {
            bool did = false;
            // ---- a batch's size is published the moment all its workers have posted theirs, whatever the state of
            //      the batches before it: other blocks wait for nothing but the packing itself ----
            const uint32_t real = ended ? handed - 1 : handed;
            if (agg_posted < real && uni32(&s_cnt[agg_posted % kRowRing]) == n_workers) {
                const uint32_t r = agg_posted % kRowRing;
                __threadfence_block();
                if (lane == 0) s_cnt[r] = 0;
                uint32_t v = lane < n_workers ? vol32(&s_tot[r][lane]) : 0u;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
                const EncItem& I = item(vol32(&s_tensor[r]));
                const uint32_t b = vol32(&s_ticket[r]) - I.first_batch;
                if (b != 0 && lane == 0) st_flag(&C.flags[I.first_batch + b], kFlagAggregate | v);
                ++agg_posted;
                if (lane == 0) *reinterpret_cast<volatile uint32_t*>(&s_agg_seq) = agg_posted;
                did = true;
            }
            // ---- the block's next batch.  A ticket is taken as late as the prefetch allows (the batch the fastest worker
            //      has begun and the one after it, whose input travels): every block
            //      behind this ticket waits for its batch to be packed.  Packed batches may wait for their place up
            //      to five deep.  A batch only ever waits for batches with smaller tickets, which blocks that are
            //      running hold: the scheme does not depend on every block of the grid being resident. ----
            if (!ended && handed < uni32(&s_lead) + kRowAhead && handed < uni32(&s_off_seq) + 6) {
                if (ticket_state == 0) {
                    if (lane == 0) ticket = atomicAdd(&C.ctl->ticket, 1u);   // used one turn of the loop later
                    ticket_state = 1;
                    did = true;
                } else {
                    if (ticket_state == 1) { ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0); ticket_state = 2; }
                    const uint32_t g = ticket;
                    uint32_t t = kNoTensor, cbase = 0;
                    bool publish = true;
                    if (g < C.total_batches) {
                        if (N_ITEMS > 1)
                            while (tcur + 1 < C.n_tensors && g >= P.item[tcur + 1].first_batch) ++tcur;
                        t = tcur;
                        const EncItem& I = item(t);
                        cbase = (g - I.first_batch) * n_workers;
                        if (t != tab_tensor) {
                            if (load_next_slot(t, agg_posted)) {
                                tab_slot = (tab_slot + 1) % kTabSlots;
                                tab_tensor = t;
                            } else {
                                publish = false;
                            }
                        }
                        if (publish && g == I.first_batch) {
                            // the fixed parts of the tensor's container: code lengths, padding of the chunk offset table,
                            // tail padding of a raw body
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
                            s_tensor[handed % kRowRing] = t; s_cbase[handed % kRowRing] = cbase; s_tabslot[handed % kRowRing] = tab_slot;
                            s_ticket[handed % kRowRing] = g;
                            __threadfence_block();
                            *reinterpret_cast<volatile uint32_t*>(&s_base_seq) = handed + 1;
                        }
                        ++handed;
                        ticket_state = 0;
                        did = true;
                    }
                }
            }
            if (ended && agg_posted == handed - 1) break;
            if (uni32(&s_fail)) break;
            if (did) { idle = 0; continue; }
            if (++idle > C.spin_limit) { s_fail = 1; break; }
            __nanosleep(kRowSleep);
        }
    } else if (warp == n_workers + 1) {
        // =========================== the placer warp ===========================
        // Finds where the block's batches go.  It keeps a cursor into the tensor's row of look-back words: cur_sum =
        // size of all batches below cur_pos.  The cursor moves forward over other blocks' batches as their sizes
        // appear, whether or not this block's own batch is packed yet, so that a batch is placed the moment the
        // cursor stands at it.  The cursor starts with a look-back from the block's first batch in the tensor.
        uint32_t placed = 0, idle = 0;
        bool lb_on = false;
        unsigned long long lb_sum = 0;
        long long lb_base = 0;
        unsigned long long* lb_flags = nullptr;
        uint32_t lb_b = 0, lb_t = 0;
        uint32_t cur_t = kNoTensor, cur_pos = 0, cur_n = 0;       // the cursor: tensor, next batch, batches of the tensor
        unsigned long long cur_sum = 0;
        unsigned long long* cur_flags = nullptr;
        for (;;) {
            bool did = false;
            const uint32_t agg_posted = uni32(&s_agg_seq);
            __threadfence_block();
            if (placed < agg_posted) {
                const uint32_t r = placed % kRowRing;
                const uint32_t tj = vol32(&s_tensor[r]);
                const uint32_t bj = vol32(&s_ticket[r]) - item(tj).first_batch;
                if (cur_t != tj && !lb_on) {
                    lb_t = tj;
                    lb_flags = C.flags + item(tj).first_batch;   // the look-back stays inside the tensor
                    lb_b = bj;
                    lb_sum = 0;
                    lb_base = (long long)lb_b - 1;
                    lb_on = true;
                    did = true;
                }
                if (lb_on) {
                    bool done = lb_b == 0;
                    if (!done) {
                        // One round: 32 * kRowLook predecessors, newest first, up to the first one that already knows
                        // its prefix.  All loads of a round are in flight together.
                        unsigned long long f[kRowLook];
#pragma unroll
                        for (int k = 0; k < kRowLook; ++k) {
                            const long long idx = lb_base - 32 * k - lane;
                            f[k] = idx >= 0 ? ld_flag(&lb_flags[idx]) : kFlagPrefix;
                        }
                        unsigned long long x = 0;
                        bool found = false, stuck = false;
#pragma unroll
                        for (int k = 0; k < kRowLook; ++k) {
                            if (found || stuck) continue;
                            const uint32_t ready = __ballot_sync(0xFFFFFFFFu, (f[k] >> 62) != 0);
                            const uint32_t prefix = __ballot_sync(0xFFFFFFFFu, (f[k] >> 62) == 2);
                            const uint32_t first_prefix = prefix ? (uint32_t)__ffs(prefix) - 1 : 32u;
                            const uint32_t need = first_prefix == 32 ? 0xFFFFFFFFu : (0xFFFFFFFFu >> (31 - first_prefix));
                            if ((ready & need) != need) { stuck = true; continue; }   // keep the windows before this one
                            if (lane <= first_prefix || first_prefix == 32) x += f[k] & kFlagValue;
                            found = first_prefix != 32;
                            if (!found) lb_base -= 32;
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
                        if (x || found) did = true;
                        lb_sum += x;
                        done = found;
                    }
                    if (done) {
                        cur_t = lb_t; cur_pos = lb_b; cur_sum = lb_sum; cur_flags = lb_flags;
                        const uint32_t next_first = (N_ITEMS > 1 && lb_t + 1 < C.n_tensors) ? P.item[N_ITEMS > 1 ? lb_t + 1 : 0].first_batch : C.total_batches;
                        cur_n = next_first - item(lb_t).first_batch;
                        lb_on = false;
                        did = true;
                    }
                }
                if (cur_t == tj && cur_pos == bj) {
                    const uint32_t v = lane < n_workers ? vol32(&s_tot[r][lane]) : 0u;
                    uint32_t inc = v;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t x = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                        if (lane >= (uint32_t)o) inc += x;
                    }
                    const uint32_t own = __shfl_sync(0xFFFFFFFFu, inc, 31);
                    if (lane == 0) st_flag(&cur_flags[bj], kFlagPrefix | (cur_sum + own));
                    // every worker learns where its chunk goes and sends its piece off itself
                    if (lane < n_workers) s_off[r][lane] = cur_sum + inc - v;
                    __threadfence_block();
                    __syncwarp();
                    if (lane == 0) *reinterpret_cast<volatile uint32_t*>(&s_off_seq) = placed + 1;
                    cur_sum += own;
                    ++cur_pos;
                    ++placed;
                    did = true;
                }
            }
            // ---- the cursor moves on over the sizes that have been published, up to this block's next batch ----
            const uint32_t handed = uni32(&s_base_seq);
            __threadfence_block();
            const bool next_known = placed < handed;             // the batch after the placed ones has been dealt out
            const uint32_t next_t = next_known ? vol32(&s_tensor[placed % kRowRing]) : kNoTensor;
            if (next_known && next_t == kNoTensor) break;         // that was the block's last batch
            if (cur_t != kNoTensor && !lb_on) {
                uint32_t stop = cur_n;
                if (next_known && next_t == cur_t) stop = vol32(&s_ticket[placed % kRowRing]) - item(cur_t).first_batch;
                if (cur_pos < stop) {
                    unsigned long long f[kRowLook];
#pragma unroll
                    for (int k = 0; k < kRowLook; ++k) {
                        const uint32_t idx = cur_pos + 32 * k + lane;
                        f[k] = idx < stop ? ld_flag(&cur_flags[idx]) : 0ull;
                    }
                    bool open = true;
#pragma unroll
                    for (int k = 0; k < kRowLook; ++k) {
                        if (!open) continue;
                        const uint32_t ready = __ballot_sync(0xFFFFFFFFu, (f[k] >> 62) != 0);
                        const uint32_t run = ready == 0xFFFFFFFFu ? 32u : (uint32_t)__ffs(~ready) - 1;   // words in a row that are there
                        if (run) {
                            const uint32_t in_run = run == 32 ? 0xFFFFFFFFu : ((1u << run) - 1);
                            const uint32_t prefix = __ballot_sync(0xFFFFFFFFu, (f[k] >> 62) == 2) & in_run;
                            const uint32_t last_prefix = prefix ? 31u - (uint32_t)__clz(prefix) : 32u;   // jump to the newest known prefix
                            unsigned long long x = 0;
                            if (lane < run && (last_prefix == 32 ? true : lane >= last_prefix)) x = f[k] & kFlagValue;
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
                            cur_sum = (last_prefix == 32 ? cur_sum : 0ull) + x;
                            cur_pos += run;
                            did = true;
                        }
                        open = run == 32;
                    }
                }
            }
            if (uni32(&s_fail)) break;
            if (did) { idle = 0; continue; }
            if (++idle > C.spin_limit) { s_fail = 1; break; }
            __nanosleep(kRowSleep);
        }
    } else {
        // =========================== a worker warp ===========================
        auto wait_seq = [&](const uint32_t* word, const uint32_t target) -> bool {
            bool ok = false;
            for (uint32_t n = 0; n < C.spin_limit; ++n) {
                if (vol32(word) >= target) { ok = true; break; }
                if (vol32(&s_fail)) break;
                if (n > 2) __nanosleep(kRowSleep);
            }
            __threadfence_block();
            return __all_sync(0xFFFFFFFFu, ok);
        };
        const uint32_t in_s = smem_u32(warp_base);
        const uint32_t pack1_s = in_s + RP.n_buf * RP.in_bytes;
        const uint32_t ring_s = pack1_s + RP.pack1_bytes;
        const uint32_t RS = RP.row_stride, U = RP.units;
        const uint32_t pack1_stride = C.sub + C.sub / 2 + 4;

        // requests the input of the block's batch `j` for this warp into buffer j & 1
        auto request = [&](const uint32_t j) {
            const uint32_t t = vol32(&s_tensor[j % kRowRing]);
            if (t != kNoTensor) {
                const EncItem& I = item(t);
                const uint32_t c = vol32(&s_cbase[j % kRowRing]) + warp;
                if (c < I.n_chunks) {
                    const uint64_t lo = (uint64_t)c * C.chunk_bytes;
                    const uint8_t* src = I.in + lo;
                    const uint64_t left = I.input_bytes - lo;           // > 0
                    const uint32_t have = (uint32_t)min((uint64_t)C.chunk_bytes, left);
                    const uint32_t buf = in_s + (j & (RP.n_buf - 1)) * RP.in_bytes;
                    // unit q = 16 bytes at offset 16 q of the chunk -> row q / U, column q % U
                    uint32_t row = lane / U, col = lane % U;
                    const uint32_t drow = 32 / U, dcol = 32 % U;
                    for (uint32_t q = lane; q < 32 * U; q += 32) {
                        const uint32_t off = 16 * q;
                        const uint32_t n = off < have ? min(16u, have - off) : 0u;
                        cp_async16(buf + row * RS + 16 * col, n ? src + off : src, n);   // bytes that do not exist read as zero
                        row += drow; col += dcol;
                        if (col >= U) { col -= U; ++row; }
                    }
                }
            }
            cp_async_commit();
        };

        uint32_t bad = 0;
        uint32_t ring_head = 0;                                   // next free 16-byte unit of the ring (mod ring size)
        uint32_t ring_used = 0;                                   // units allocated and not yet known to be free
        uint32_t ring_sent = 0;                                   // of which: units whose copies have been issued
        const uint32_t ring_units = RP.ring_bytes / 16;
        bool failed = false;
        uint32_t sent = 0;                                        // batches of this block whose piece this warp has sent off
        // Chunks this warp has sent off, per tensor; added to the tensor's counters when the warp moves on to
        // another tensor or leaves.  Whoever completes a tensor writes its header.
        uint32_t acc_t = kNoTensor, acc_n = 0;
        unsigned long long acc_bits0 = 0, acc_bits1 = 0;
        auto flush_acc = [&]() {                                  // lane 0
            if (acc_n == 0) return;
            TensorCounters* tc = counters(acc_t);
            if (H0) atomicAdd(&tc->payload_bits[0], acc_bits0);
            if (H1) atomicAdd(&tc->payload_bits[1], acc_bits1);
            __threadfence();
            const uint32_t before = atomicAdd(&tc->done, acc_n);
            if (before + acc_n == item(acc_t).n_chunks) {
                __threadfence();
                write_header(C, item(acc_t), tc);
            }
            acc_n = 0;
            acc_bits0 = acc_bits1 = 0;
        };
        // Sends off the pieces of all batches below `upto` that have been placed by now (lane 0 does the work: one
        // bulk copy shared -> global per piece, two when the piece wraps around the ring, and the chunk's table entries).
        auto send_placed = [&](const uint32_t upto) {
            const uint32_t placed_now = min(uni32(&s_off_seq), upto);
            if (sent >= placed_now) return;
            __threadfence_block();
            if (lane == 0) {
                for (; sent < placed_now; ++sent) {
                    const uint32_t r = sent % kRowRing;
                    const uint32_t t = vol32(&s_tensor[r]);
                    const EncItem& I = item(t);
                    const uint32_t c = vol32(&s_cbase[r]) + warp;
                    if (c >= I.n_chunks) continue;
                    const unsigned long long off16 = *reinterpret_cast<const volatile unsigned long long*>(&s_off[r][warp]);
                    const uint32_t tot = vol32(&s_tot[r][warp]), p0 = vol32(&s_p0[r][warp]);
                    uint32_t hs = 0;
#pragma unroll
                    for (int s = 0; s < 2; ++s) {
                        if (!is_huff(s)) continue;
                        reinterpret_cast<uint32_t*>(I.out + I.lay.chunk_off_tab[s])[c] = (uint32_t)(off16 + (hs ? p0 : 0u));
                        ++hs;
                    }
                    if (tot) {
                        uint8_t* dst = I.out + I.lay.payload_off + 16 * off16;
                        const uint32_t ro = 16 * vol32(&s_roff[r][warp]), len = 16 * tot;
                        const uint32_t first = min(len, RP.ring_bytes - ro);
                        bulk_s2g(dst, ring_s + ro, first);
                        if (first < len) bulk_s2g(dst + first, ring_s, len - first);
                        ring_sent += tot;
                    }
                    if (c == I.n_chunks - 1) counters(t)->total16 = off16 + tot;
                    if (t != acc_t) { flush_acc(); acc_t = t; }
                    ++acc_n;
                    acc_bits0 += *reinterpret_cast<const volatile uint16_t*>(&s_bits[r][warp][0]);
                    acc_bits1 += *reinterpret_cast<const volatile uint16_t*>(&s_bits[r][warp][1]);
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            sent = __shfl_sync(0xFFFFFFFFu, sent, 0);
            ring_sent = __shfl_sync(0xFFFFFFFFu, ring_sent, 0);
        };
        uint32_t requested = 0;                                   // batches whose input has been requested
        for (uint32_t it = 0;; ++it) {
            // (a batch whose input has been requested has been seen already; no second wait, and above all no memory
            // fence while the asynchronous copies are in flight: the fence would wait for them)
            if (requested <= it && !wait_seq(&s_base_seq, it + 1)) { failed = true; break; }
            if (lane == 0 && vol32(&s_lead) < it + 1) atomicMax(&s_lead, it + 1);
            const uint32_t t = vol32(&s_tensor[it % kRowRing]);
            if (t == kNoTensor) {
                // everything this warp packed must leave before the block's shared memory goes away
                for (uint32_t n = 0; n < C.spin_limit && sent < it; ++n) {
                    send_placed(it);
                    if (sent < it) { if (uni32(&s_fail)) break; __nanosleep(200); }
                }
                if (sent < it) failed = true;
                break;
            }
            if (requested <= it) { request(it); requested = it + 1; }
            cp_async_wait_all();
            __syncwarp();
            // two buffers: the next batch's input travels while this one is packed (if it has been dealt out already)
            if (RP.n_buf == 2 && uni32(&s_base_seq) >= it + 2) { __threadfence_block(); request(it + 1); requested = it + 2; }

            const EncItem& I = item(t);
            const uint32_t my_c = vol32(&s_cbase[it % kRowRing]) + warp;
            const bool active = my_c < I.n_chunks;
            const uint64_t c_lo = (uint64_t)(active ? my_c : 0) * C.cs;
            const uint32_t c_syms = active ? (uint32_t)min((uint64_t)C.cs, I.n_syms - c_lo) : 0u;
            const uint32_t lo_sym = lane * C.sub;
            const uint32_t n_my = lo_sym < c_syms ? min(C.sub, c_syms - lo_sym) : 0u;
            const uint32_t tab_slot_idx = vol32(&s_tabslot[it % kRowRing]);
            const uint32_t tab_s = smem_u32(tabs + tab_slot_idx * tab_words);
            const uint32_t row_s = in_s + (it & (RP.n_buf - 1)) * RP.in_bytes + lane * RS;
            const uint32_t p1_s = pack1_s + lane * pack1_stride;

            // ---- pack: 16 input bytes = 8 symbols of each stream at a time ----
            uint32_t hi0 = 0, nb0 = 0, w0 = row_s, hi1 = 0, nb1 = 0, w1 = (H0 && H1) ? p1_s : row_s;
            uint32_t seen = 0;
            uint8_t* const raw0 = I.out + I.lay.section_off[0] + c_lo + lo_sym;     // this lane's bytes of a raw stream
            uint8_t* const raw1 = I.out + I.lay.section_off[1] + c_lo + lo_sym;
            auto emit4 = [&](const uint32_t four, const uint32_t tab, uint32_t& hi, uint32_t& nb, uint32_t& waddr) {
                const uint32_t e0 = lds32(tab + 4u * __byte_perm(four, 0, 0x4440));
                const uint32_t e1 = lds32(tab + 4u * __byte_perm(four, 0, 0x4441));
                const uint32_t e2 = lds32(tab + 4u * __byte_perm(four, 0, 0x4442));
                const uint32_t e3 = lds32(tab + 4u * __byte_perm(four, 0, 0x4443));
                seen |= e0 | e1 | e2 | e3;
                const uint32_t ca = (e0 | __funnelshift_r(e1, 0, e0)) & 0xFFFFFF00u;
                put_bits_row(ca, (e0 + e1) & 31, hi, nb, waddr);
                const uint32_t cb = (e2 | __funnelshift_r(e3, 0, e2)) & 0xFFFFFF00u;
                put_bits_row(cb, (e2 + e3) & 31, hi, nb, waddr);
            };
            const uint32_t full_units = n_my / 8;
            uint32_t keep[4] = {0, 0, 0, 0};                       // raw bytes of two units: one 16-byte store
            for (uint32_t u = 0; u < full_units; ++u) {
                const uint4 x = lds128e(row_s + 16 * u);
                const uint32_t w[4] = {x.x, x.y, x.z, x.w};
                uint32_t sy[2][2];
                split16<FMT>(w, sy[0], sy[1]);
                if (H0) { emit4(sy[0][0], tab_s, hi0, nb0, w0); emit4(sy[0][1], tab_s, hi0, nb0, w0); }
                if (H1) { emit4(sy[1][0], tab_s + (H0 ? 1024 : 0), hi1, nb1, w1); emit4(sy[1][1], tab_s + (H0 ? 1024 : 0), hi1, nb1, w1); }
                if (!H0 || !H1) {
                    const uint32_t* r = H0 ? sy[1] : sy[0];
                    if (u & 1) st_cs_v4((H0 ? raw1 : raw0) + 8 * (u - 1), make_uint4(keep[0], keep[1], r[0], r[1]));
                    else { keep[0] = r[0]; keep[1] = r[1]; }
                }
            }
            // ragged end of the tensor's last chunk: the lane's last, incomplete unit (missing bytes were read as zero)
            const uint32_t tail = n_my - 8 * full_units;
            if (tail || ((full_units & 1) && (!H0 || !H1))) {
                uint32_t sy[2][2] = {{0, 0}, {0, 0}};
                if (tail) {
                    const uint4 x = lds128e(row_s + 16 * full_units);
                    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
                    split16<FMT>(w, sy[0], sy[1]);
#pragma unroll
                    for (int s = 0; s < 2; ++s) {
                        if (!is_huff(s)) continue;
                        const uint32_t tab = tab_s + ((s == 1 && H0) ? 1024 : 0);
                        for (uint32_t i = 0; i < tail; ++i) {
                            const uint32_t sym = (sy[s][i >> 2] >> (8 * (i & 3))) & 0xFF;
                            const uint32_t e = lds32(tab + 4 * sym);
                            seen |= e;
                            if (s == 0) put_bits_row(e & 0xFFFFFF00u, e & 31, hi0, nb0, w0);
                            else put_bits_row(e & 0xFFFFFF00u, e & 31, hi1, nb1, w1);
                        }
                    }
                }
                if (!H0 || !H1) {
                    // the raw stream's last bytes of this lane: whole 8-byte halves that hold symbols (the body is
                    // padded to 16 bytes, which the service warp of the tensor's first batch clears)
                    const uint32_t* r = H0 ? sy[1] : sy[0];
                    uint8_t* dst = (H0 ? raw1 : raw0) + 8 * (full_units & ~1u);
                    if (full_units & 1) {
                        st_cs_v2(dst, make_uint2(keep[0], keep[1]));
                        if (tail) st_cs_v2(dst + 8, make_uint2(r[0], r[1]));
                    } else if (tail) {
                        st_cs_v2(dst, make_uint2(r[0], r[1]));
                    }
                }
            }
            if (H0 && n_my) sts32(w0, hi0);                       // pending bits (or zero)
            if (H1 && n_my) sts32(w1, hi1);
            if (seen & 16) bad = t + 1;                            // an entry without a code carries bit 4
            uint32_t my_bits[2] = {0, 0};
            if (H0) my_bits[0] = 8 * (w0 - row_s) + nb0;
            if (H1) my_bits[1] = 8 * (w1 - ((H0 && H1) ? p1_s : row_s)) + nb1;
            __syncwarp();

            // ---- subchunk end bits and the sizes of the chunk's pieces ----
            uint32_t end[2] = {0, 0}, piece16[2] = {0, 0}, cbits[2] = {0, 0};
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
                    uint32_t chunk_bits = __shfl_sync(0xFFFFFFFFu, inc, 31);
                    // A chunk that holds nothing but the fill symbol (the symbol with the all-zero code, the shortest
                    // one) takes no bits at all.  Such a chunk has exactly symbols * length bits (rare otherwise), and
                    // all of them are zero: every other code has a one somewhere.
                    {
                        const uint32_t fill_len = vol32(&s_fill[tab_slot_idx][hs]) >> 8;
                        if (active && chunk_bits == c_syms * fill_len) {
                            const uint32_t src = (s == 1 && H0) ? p1_s : row_s;
                            uint32_t any = 0;
                            for (uint32_t i = 0; i < (my_bits[s] + 31) / 32; ++i) any |= lds32(src + 4 * i);
                            if (!__any_sync(0xFFFFFFFFu, any != 0)) { inc = 0; chunk_bits = 0; }
                        }
                    }
                    end[s] = inc; cbits[s] = chunk_bits;
                    if (active) {
                        if (C.sub_width == 2) reinterpret_cast<uint16_t*>(I.out + I.lay.sub_end_tab[s] + 64ull * my_c)[lane] = (uint16_t)inc;
                        else reinterpret_cast<uint32_t*>(I.out + I.lay.sub_end_tab[s] + 128ull * my_c)[lane] = inc;
                        piece16[s] = (chunk_bits + 127) / 128;
                    }
                    ++hs;
                }
            }
            const uint32_t need = piece16[0] + piece16[1];

            // ---- room in the ring: give back what the service warp has sent off, wait if that is not enough ----
            uint32_t roff = ring_head;
            if (need) {
                bool room = false;
                for (uint32_t n = 0; n < C.spin_limit; ++n) {
                    if (ring_used + need <= ring_units) { room = true; break; }
                    // pieces that have been sent are free as soon as their copies have read them
                    send_placed(it);
                    if (ring_sent) {
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        __syncwarp();
                        ring_used -= ring_sent;
                        ring_sent = 0;
                        continue;
                    }
                    if (uni32(&s_fail)) break;
                    __nanosleep(kRowSleep);
                }
                if (!room) { failed = true; break; }
                ring_head = (ring_head + need) % ring_units;
                ring_used += need;
            }
            // ---- every lane moves its bits to their place in the piece ----
            {
                uint32_t piece_word = 4 * roff;                                   // first word of the piece in the ring
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    if (!is_huff(s)) continue;
                    const uint32_t e = end[s];
                    uint32_t start = __shfl_up_sync(0xFFFFFFFFu, e, 1);
                    if (lane == 0) start = 0;
                    const uint32_t bits = e - start;
                    const uint32_t chunk_bits = cbits[s];
                    const uint32_t piece_words = 4 * piece16[s];
                    const uint32_t src = (s == 1 && H0) ? p1_s : row_s;
                    const uint32_t sh = start & 31, d0 = start >> 5;
                    const uint32_t n_dst = (sh + bits + 31) / 32, n_src = (bits + 31) / 32;
                    auto dst = [&](const uint32_t w) { return ring_s + 4 * ((piece_word + w) & (ring_words - 1)); };
                    if (piece_words) {
                        if (__all_sync(0xFFFFFFFFu, bits >= 32)) {
                            // every lane spans a word boundary, so a destination word is shared by at most two
                            // neighbouring lanes: a lane hands its ragged last word to the next lane
                            const bool ragged = ((sh + bits) & 31) != 0;
                            const uint32_t il = n_dst - 1;
                            const uint32_t lc = il < n_src ? lds32(src + 4 * il) : 0u;
                            const uint32_t lp = il >= 1 ? lds32(src + 4 * (il - 1)) : 0u;
                            const uint32_t tailw = ragged ? __funnelshift_r(lc, lp, sh) : 0u;
                            uint32_t head = __shfl_up_sync(0xFFFFFFFFu, tailw, 1);
                            if (lane == 0) head = 0;
                            const uint32_t n_mine = n_dst - ((ragged && lane != 31) ? 1u : 0u);
                            uint32_t prev = 0;
                            for (uint32_t i = 0; i < n_mine; ++i) {
                                const uint32_t cur = i < n_src ? lds32(src + 4 * i) : 0u;
                                uint32_t v = __funnelshift_r(cur, prev, sh);      // (prev:cur) >> sh, low word
                                prev = cur;
                                if (i == 0) v |= head;
                                sts32(dst(d0 + i), v);
                            }
                            if (lane < 4) {                                       // zero padding up to the 16-byte boundary
                                const uint32_t w = piece_words - 4 + lane;
                                if (32 * w >= chunk_bits) sts32(dst(w), 0);
                            }
                        } else {
                            // general case (short or empty subchunks): the piece starts from zero and is OR-ed into
                            for (uint32_t w = lane; w < piece_words; w += 32) sts32(dst(w), 0);
                            __syncwarp();
                            uint32_t prev = 0;
                            for (uint32_t i = 0; i < n_dst && bits; ++i) {
                                const uint32_t cur = i < n_src ? lds32(src + 4 * i) : 0u;
                                const uint32_t v = __funnelshift_r(cur, prev, sh);
                                prev = cur;
                                asm volatile("red.shared.or.b32 [%0], %1;" :: "r"(dst(d0 + i)), "r"(v) : "memory");
                            }
                        }
                    }
                    piece_word += piece_words;
                }
            }
            // what the lanes wrote must be visible to the bulk copy that reads it
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                const uint32_t r = it % kRowRing;
                s_tot[r][warp] = need; s_p0[r][warp] = piece16[0]; s_roff[r][warp] = roff;
                s_bits[r][warp][0] = (uint16_t)cbits[0]; s_bits[r][warp][1] = (uint16_t)cbits[1];
                __threadfence_block();
                atomicAdd(&s_cnt[r], 1u);
            }
            // pieces of earlier batches that have been placed leave now (before the next input is requested: the
            // fences on this path would wait for the copies in flight)
            __syncwarp();
            send_placed(it);
            // one buffer: the rows are free now, the next batch's input travels while this warp waits
            if (RP.n_buf == 1 && uni32(&s_base_seq) >= it + 2) { __threadfence_block(); request(it + 1); requested = it + 2; }
        }
        if (lane == 0) {
            flush_acc();
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        }
        if (failed) s_fail = 1;
        if (bad && raise_status(C.ctl, 0, ZC_E_NO_CODE)) C.ctl->failed = item(bad - 1).index + 1;
    }
    __syncthreads();
    if (s_fail && threadIdx.x == 0) raise_status(C.ctl, 0, ZC_E_DEVICE_TIMEOUT);
}

}  // namespace zc
