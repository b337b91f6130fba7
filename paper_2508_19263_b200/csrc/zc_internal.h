// Internal definitions shared by the host logic and the kernels of libzc.
#pragma once
#include <stdint.h>
#include <stddef.h>
#include "zc.h"

namespace zc {

constexpr uint32_t kLmax = 12;            // longest code; decode table has 2^12 entries
constexpr uint32_t kSubs = 32;            // subchunks per chunk = lanes of the decoding warp
constexpr uint32_t kHeaderBytes = 128;
constexpr uint32_t kMagic = 0x3031435Au;  // 'Z','C','1','0' little-endian

// Byte offsets inside the 128-byte header.
constexpr uint32_t kHdrMagic = 0, kHdrVersion = 4, kHdrFormat = 6, kHdrStreams = 7, kHdrElems = 8,
                   kHdrChunkBytes = 16, kHdrChunks = 20, kHdrLmax = 24, kHdrGroup = 25, kHdrSubs = 26, kHdrSubWidth = 27,
                   kHdrTotal = 32, kHdrPayloadOff = 40, kHdrPayloadBytes = 48, kHdrStream0 = 64,
                   kHdrStreamStride = 32;
// Inside a stream descriptor.
constexpr uint32_t kSdMode = 0, kSdSyms = 8, kSdBits = 16, kSdSection = 24;

inline uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

// Where things are for given modes: everything except the payload size is known before encoding.
struct Layout {
    uint64_t section_off[2];   // table section (HUFF) or raw body (RAW)
    uint64_t chunk_off_tab[2]; // HUFF: offset of chunk_off16[]
    uint64_t sub_end_tab[2];   // HUFF: offset of sub_end[][32]
    uint64_t payload_off;
};

}  // namespace zc

struct zc_plan_s {
    uint32_t format, group, chunk_bytes, n_chunks;
    uint64_t n_elems, n_syms, input_bytes;
    uint32_t syms_per_chunk, syms_per_sub;
};

struct zc_codebook_s {
    uint32_t mode[2];
    uint8_t len[2][256];
    uint32_t code[2][256];     // right-aligned canonical code values
    // derived once when the codebook is built, so that a compress call only copies them:
    uint32_t enc[2][256];      // the encoder's table entry of every symbol: code << (32 - length) | length; 16: no code
    uint8_t wide[2];           // the stream's codes are long on average: the encoder uses 12-bit pack slots
    uint8_t brief[2];          // the stream's codes are short on average: half-size pack slots do for long subchunks
};

namespace zc {
// Fills the derived fields of a codebook (call after len[] and code[] are final).
// wide: with the symbol probabilities the code lengths imply (2^-length) the expected length is above 6.5 bits;
// brief: it is at most 3.25 bits.
inline void finish_codebook(zc_codebook_s* cb)
{
    for (int s = 0; s < 2; ++s) {
        uint64_t acc = 0;                        // sum of length * 2^(12 - length)
        for (int v = 0; v < 256; ++v) {
            const uint32_t l = cb->len[s][v];
            cb->enc[s][v] = l ? (cb->code[s][v] << (32 - l)) | l : 16u;
            if (l) acc += (uint64_t)l << (12 - l);
        }
        cb->wide[s] = 2 * acc > (13ull << 12) ? 1 : 0;
        cb->brief[s] = 4 * acc <= (13ull << 12) ? 1 : 0;
    }
}


// Bytes of one sub_end entry: chunks of at most 8 KiB hold fewer than 65536 bits, so 16 bits are enough.
inline uint32_t sub_end_width(uint32_t chunk_bytes) { return chunk_bytes <= 8192 ? 2u : 4u; }

inline uint64_t table_section_bytes(uint32_t n_chunks, uint32_t chunk_bytes)
{
    return 256 + round_up(4ull * n_chunks, 16) + 32ull * sub_end_width(chunk_bytes) * n_chunks;
}

inline Layout make_layout(const zc_plan_s& p, const uint32_t mode[2])
{
    Layout L{};
    uint64_t off = kHeaderBytes;
    for (int s = 0; s < 2; ++s)
        if (mode[s] == ZC_MODE_HUFF) {
            L.section_off[s] = off;
            L.chunk_off_tab[s] = off + 256;
            L.sub_end_tab[s] = off + 256 + round_up(4ull * p.n_chunks, 16);
            off += table_section_bytes(p.n_chunks, p.chunk_bytes);
        }
    for (int s = 0; s < 2; ++s)
        if (mode[s] == ZC_MODE_RAW) {
            L.section_off[s] = off;
            off += round_up(p.n_syms, 16);
        }
    L.payload_off = off;
    return L;
}

// What the encoder accumulates per tensor on the device.
struct TensorCounters {
    unsigned long long payload_bits[2];
    unsigned long long total16;  // payload area size in 16-byte units
    uint32_t done;               // chunks that are completely written
    uint32_t pad;
};

// Device workspace: a control block, then whatever the call needs behind it (zc_compress: one look-back
// word per chunk).
struct Control {
    unsigned long long status;   // (call id << 8) | zc_status raised on the device; first error of a call wins
    unsigned long long call_id;  // id of the call that last used the block; a status with another id is stale.
                                 // The compress calls clear the whole block and use id 0.
    uint32_t ticket;             // next batch of chunks (encoder) or range of chunks (batched decoder) to hand out
    uint32_t failed;             // batched calls: 1 + index of the tensor the recorded error belongs to
    TensorCounters tc;           // zc_compress: the counters of its one tensor
    uint32_t pad[4];
};
constexpr size_t kControlBytes = 256;

// What the test hooks (zc_test_hooks.h) can change; the product path never writes these.
struct TestKnobs {
    uint32_t spin_limit;     // polls after which a bounded wait on the device gives up
    uint32_t first_ticket;   // first batch the encoder hands out (not 0: batch 0 is never packed, so every look-back stalls)
    uint32_t skip_copy;      // the decoder does not start the copies of the pieces it then waits for
};
TestKnobs& test_knobs();
// Development build (-DZC_DEBUG_CHECKS=1): each translation unit with kernels adds its counts of refused shared and
// global accesses to out[0] and out[1] and clears them; in the ordinary build they do nothing.
void debug_counts_hist(uint32_t out[2]);
void debug_counts_encode(uint32_t out[2]);
void debug_counts_decode(uint32_t out[2]);
constexpr uint32_t kDefaultSpinLimit = 1u << 22;

}  // namespace zc
