// Word-level field split and merge for the three element formats.
//
// In every format 4 bytes of elements carry exactly 2 symbols of each stream, and 16 bytes
// carry 8.  split_word() turns one 32-bit input word into the two exponent symbols and the two
// sign+mantissa symbols it contains, each pair returned "spread": first symbol in byte 0, second
// in byte 2.  merge_word() is the inverse.  pack_spread()/spread_lo()/spread_hi() move between
// the spread form and 4 symbols packed in a word.  All of it is plain 32-bit logic so that one
// thread handles 8 symbols per 16-byte load.
#pragma once
#include <stdint.h>
#include "zc.h"

#if defined(__CUDACC__)
#define ZC_HD __host__ __device__ __forceinline__
#else
#define ZC_HD inline
#endif

namespace zc {

// Byte permute with the semantics of PRMT's default mode: selector nibble k picks byte k of the
// 8-byte pool {a (bytes 0-3), b (bytes 4-7)}.
ZC_HD uint32_t byte_perm(uint32_t a, uint32_t b, uint32_t sel)
{
#if defined(__CUDA_ARCH__)
    return __byte_perm(a, b, sel);
#else
    const uint64_t pool = ((uint64_t)b << 32) | a;
    uint32_t r = 0;
    for (int k = 0; k < 4; ++k) r |= (uint32_t)((pool >> (8 * ((sel >> (4 * k)) & 7))) & 0xFF) << (8 * k);
    return r;
#endif
}

// x * 128 as a multiply-add, so that it does not compete with the shifts and logic ops for the integer pipe
ZC_HD uint32_t mul128(uint32_t x)
{
#if defined(__CUDA_ARCH__)
    uint32_t r;
    asm("mad.lo.u32 %0, %1, 128, 0;" : "=r"(r) : "r"(x));
    return r;
#else
    return x * 128u;
#endif
}

// two spread pairs -> 4 packed symbols (bytes 0,2 of a then bytes 0,2 of b)
ZC_HD uint32_t pack_spread(uint32_t a, uint32_t b) { return byte_perm(a, b, 0x6420); }
// 4 packed symbols -> spread pair of symbols 0,1 / of symbols 2,3 (bytes 1 and 3 are zero)
ZC_HD uint32_t spread_lo(uint32_t p) { return byte_perm(p, 0, 0x4140); }
ZC_HD uint32_t spread_hi(uint32_t p) { return byte_perm(p, 0, 0x4342); }

template <int FMT> struct Fields;

// Scale bytes have no fields: split16 / merge16 handle them whole (the word-level pair is never used).
template <> struct Fields<ZC_FMT_SCALE_U8> {
    static ZC_HD void split_word(uint32_t, uint32_t& e, uint32_t& sm) { e = 0; sm = 0; }
    static ZC_HD uint32_t merge_word(uint32_t, uint32_t) { return 0; }
};

// BF16: two elements per word; exponent = bits 14..7, sign+mantissa = (bit 15 -> bit 7) | bits 6..0.
template <> struct Fields<ZC_FMT_BF16> {
    static ZC_HD void split_word(uint32_t v, uint32_t& e, uint32_t& sm)
    {
        e = (v >> 7) & 0x00FF00FFu;
        const uint32_t t = v & 0x807F807Fu;
        sm = (t | (t >> 8)) & 0x00FF00FFu;
    }
    static ZC_HD uint32_t merge_word(uint32_t e, uint32_t sm)
    {
        return (e << 7) | (sm & 0x007F007Fu) | ((sm & 0x00800080u) << 8);
    }
};

// FP8 E4M3: four elements per word; a symbol holds two 4-bit fields, lower element in the low nibble.
template <> struct Fields<ZC_FMT_FP8_E4M3> {
    static ZC_HD void split_word(uint32_t v, uint32_t& e, uint32_t& sm)
    {
        const uint32_t ev = (v >> 3) & 0x0F0F0F0Fu;
        e = (ev | (ev >> 4)) & 0x00FF00FFu;
        const uint32_t sv = ((v >> 4) & 0x08080808u) | (v & 0x07070707u);
        sm = (sv | (sv >> 4)) & 0x00FF00FFu;
    }
    static ZC_HD uint32_t merge_word(uint32_t e, uint32_t sm)
    {
        const uint32_t ex = (e | (e << 4)) & 0x0F0F0F0Fu;
        const uint32_t sx = (sm | (sm << 4)) & 0x0F0F0F0Fu;
        return (ex << 3) | (sx & 0x07070707u) | ((sx & 0x08080808u) << 4);
    }
};

// FP4 E2M1: eight elements per word (two per byte, even element in the low nibble); a symbol
// holds four 2-bit fields, lowest element in bits 1..0.
template <> struct Fields<ZC_FMT_FP4_E2M1> {
    static ZC_HD uint32_t squeeze(uint32_t x)   // 2-bit field per nibble -> four fields per byte, spread
    {
        const uint32_t t = (x | (x >> 2)) & 0x0F0F0F0Fu;
        return (t | (t >> 4)) & 0x00FF00FFu;
    }
    static ZC_HD uint32_t expand(uint32_t s)    // inverse of squeeze
    {
        const uint32_t x = (s | (s << 4)) & 0x0F0F0F0Fu;
        return (x | (x << 2)) & 0x33333333u;
    }
    static ZC_HD void split_word(uint32_t v, uint32_t& e, uint32_t& sm)
    {
        e = squeeze((v >> 1) & 0x33333333u);
        sm = squeeze(((v >> 2) & 0x22222222u) | (v & 0x11111111u));
    }
    static ZC_HD uint32_t merge_word(uint32_t e, uint32_t sm)
    {
        const uint32_t ey = expand(e), sy = expand(sm);
        return (ey << 1) | (sy & 0x11111111u) | ((sy & 0x22222222u) << 2);
    }
};

// 16 bytes of elements -> 8 exponent symbols (e[0] = symbols 0..3, e[1] = 4..7) and 8 sign+mantissa symbols.
template <int FMT>
ZC_HD void split16(const uint32_t in[4], uint32_t e[2], uint32_t sm[2])
{
    if (FMT == ZC_FMT_SCALE_U8) {
        // scale bytes: odd offsets are stream 0, even offsets stream 1
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            e[h] = byte_perm(in[2 * h], in[2 * h + 1], 0x7531);
            sm[h] = byte_perm(in[2 * h], in[2 * h + 1], 0x6420);
        }
        return;
    }
    if (FMT == ZC_FMT_BF16) {
        // gather the four high bytes (sign, exponent bits 7..1) and the four low bytes (exponent bit 0,
        // mantissa) of four elements, then recombine per byte lane
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t hb = byte_perm(in[2 * h], in[2 * h + 1], 0x7531);
            const uint32_t lb = byte_perm(in[2 * h], in[2 * h + 1], 0x6420);
            sm[h] = (lb & 0x7F7F7F7Fu) | (hb & 0x80808080u);
            e[h] = ((hb << 1) & 0xFEFEFEFEu) | ((lb >> 7) & 0x01010101u);
        }
        return;
    }
    if (FMT == ZC_FMT_FP8_E4M3) {
        // gather the even elements (low nibbles of the symbols) and the odd ones (high nibbles) of eight bytes,
        // then build four symbols of each stream with per-byte-lane logic
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t ev = byte_perm(in[2 * h], in[2 * h + 1], 0x6420);
            const uint32_t od = byte_perm(in[2 * h], in[2 * h + 1], 0x7531);
            e[h] = ((ev >> 3) & 0x0F0F0F0Fu) | ((od << 1) & 0xF0F0F0F0u);
            const uint32_t lo = ((ev >> 4) & 0x08080808u) | (ev & 0x07070707u);
            const uint32_t hi = (od & 0x80808080u) | ((od << 4) & 0x70707070u);
            sm[h] = lo | hi;
        }
        return;
    }
    uint32_t ea, sa, eb, sb;
    Fields<FMT>::split_word(in[0], ea, sa);
    Fields<FMT>::split_word(in[1], eb, sb);
    e[0] = pack_spread(ea, eb);
    sm[0] = pack_spread(sa, sb);
    Fields<FMT>::split_word(in[2], ea, sa);
    Fields<FMT>::split_word(in[3], eb, sb);
    e[1] = pack_spread(ea, eb);
    sm[1] = pack_spread(sa, sb);
}

// inverse of split16
template <int FMT>
ZC_HD void merge16(const uint32_t e[2], const uint32_t sm[2], uint32_t out[4])
{
    if (FMT == ZC_FMT_SCALE_U8) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            out[2 * h] = byte_perm(sm[h], e[h], 0x5140);
            out[2 * h + 1] = byte_perm(sm[h], e[h], 0x7362);
        }
        return;
    }
    if (FMT == ZC_FMT_BF16) {
        // element = sign | exponent << 7 | mantissa.  The exponent byte goes to bits 14..7 (placed in byte 0
        // and multiplied by 128 on the multiply-add pipe); the sign+mantissa byte is duplicated into both bytes so that its bit 7
        // lands on bit 15 and its bits 6..0 on bits 6..0; one select picks each bit from the right source.
        const uint32_t m = 0x7F807F80u;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t xl = mul128(byte_perm(e[h], 0, 0x4140)), yl = byte_perm(sm[h], 0, 0x1100);
            const uint32_t xh = mul128(byte_perm(e[h], 0, 0x4342)), yh = byte_perm(sm[h], 0, 0x3322);
            out[2 * h] = (xl & m) | (yl & ~m);
            out[2 * h + 1] = (xh & m) | (yh & ~m);
        }
        return;
    }
    if (FMT == ZC_FMT_FP8_E4M3) {
        // element = sign << 7 | exponent << 3 | mantissa: the even elements come from the low nibbles of four
        // symbols, the odd ones from the high nibbles; then the two byte vectors are interleaved
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t ev = ((e[h] << 3) & 0x78787878u) | (sm[h] & 0x07070707u) | ((sm[h] << 4) & 0x80808080u);
            const uint32_t od = ((e[h] >> 1) & 0x78787878u) | ((sm[h] >> 4) & 0x07070707u) | (sm[h] & 0x80808080u);
            out[2 * h] = byte_perm(ev, od, 0x5140);
            out[2 * h + 1] = byte_perm(ev, od, 0x7362);
        }
        return;
    }
    out[0] = Fields<FMT>::merge_word(spread_lo(e[0]), spread_lo(sm[0]));
    out[1] = Fields<FMT>::merge_word(spread_hi(e[0]), spread_hi(sm[0]));
    out[2] = Fields<FMT>::merge_word(spread_lo(e[1]), spread_lo(sm[1]));
    out[3] = Fields<FMT>::merge_word(spread_hi(e[1]), spread_hi(sm[1]));
}

}  // namespace zc
