// Host logic of libzc: plans, codebooks, container checks, statistics.
// Nothing in this file touches the GPU, so it also runs on machines without one.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <thread>
#include <vector>

#include "zc_bits.cuh"
#include "zc_internal.h"
#include "zc_test_hooks.h"

using namespace zc;

namespace {

uint32_t group_of(uint32_t fmt)
{
    switch (fmt) {
    case ZC_FMT_BF16: return 1;
    case ZC_FMT_FP8_E4M3: return 2;
    case ZC_FMT_FP4_E2M1: return 4;
    case ZC_FMT_SCALE_U8: return 2;
    case ZC_FMT_FP8_E5M2: return 2;
    default: return 0;
    }
}

uint64_t rd(const uint8_t* p, int n)
{
    uint64_t v = 0;
    for (int i = 0; i < n; ++i) v |= (uint64_t)p[i] << (8 * i);
    return v;
}

// Optimal code lengths under a maximum length, by package-merge in its prefix-count form:
// only the weights and the leaf/package flags of each level's merged list are kept.  Because
// the leaves are sorted, the leaves chosen at a level are always a prefix of the sorted list,
// so a symbol's length is the number of levels whose chosen prefix reaches it.
// Order rules (they decide ties, hence the exact lengths): leaves ascending by
// (count, symbol); at equal weight a leaf is taken before a package.
bool limited_lengths(const uint64_t hist[256], uint32_t L, uint8_t len[256])
{
    std::memset(len, 0, 256);
    int order[256];
    size_t n = 0;
    for (int v = 0; v < 256; ++v)
        if (hist[v]) order[n++] = v;
    if (n == 0) return true;
    if (n == 1) { len[order[0]] = 1; return true; }
    if (L > kLmax || (1ull << L) < n) return false;
    std::sort(order, order + n, [&](int a, int b) {
        return hist[a] != hist[b] ? hist[a] < hist[b] : a < b;
    });
    uint64_t leaf_w[256];
    for (size_t i = 0; i < n; ++i) leaf_w[i] = hist[order[i]];

    // level r: merged list of the n leaves and the packages made of pairs of level r-1; a list never has
    // more than 2n - 1 items.  Only the weights are needed to build the next level, only the flags afterwards.
    static thread_local uint64_t w[2][512];
    static thread_local uint8_t leaf[kLmax][512];
    size_t size[kLmax];
    for (size_t i = 0; i < n; ++i) { w[0][i] = leaf_w[i]; leaf[0][i] = 1; }
    size[0] = n;
    for (uint32_t r = 1; r < L; ++r) {
        const uint64_t* pw = w[(r - 1) & 1];
        uint64_t* cw = w[r & 1];
        uint8_t* cf = leaf[r];
        const size_t np = size[r - 1] / 2;
        size_t a = 0, b = 0, m = 0;
        while (a < n && b < np) {
            const uint64_t pk = pw[2 * b] + pw[2 * b + 1];
            if (leaf_w[a] <= pk) { cw[m] = leaf_w[a++]; cf[m++] = 1; }
            else { cw[m] = pk; cf[m++] = 0; ++b; }
        }
        for (; a < n; ++a) { cw[m] = leaf_w[a]; cf[m++] = 1; }
        for (; b < np; ++b) { cw[m] = pw[2 * b] + pw[2 * b + 1]; cf[m++] = 0; }
        size[r] = m;
    }
    size_t take = 2 * n - 2;
    for (int r = (int)L - 1; r >= 0 && take > 0; --r) {
        if (take > size[r]) return false;
        size_t leaves = 0;
        for (size_t k = 0; k < take; ++k) leaves += leaf[r][k];
        for (size_t i = 0; i < leaves; ++i) len[order[i]]++;
        take = 2 * (take - leaves);
    }
    return true;
}

// Canonical assignment: walk the lengths from short to long, symbols ascending inside a length.
void canonical(const uint8_t len[256], uint32_t code[256])
{
    uint32_t count[kLmax + 2] = {0}, first[kLmax + 2] = {0};
    for (int v = 0; v < 256; ++v)
        if (len[v]) count[len[v]]++;
    uint32_t c = 0;
    for (uint32_t l = 1; l <= kLmax; ++l) {
        c = (c + count[l - 1]) << 1;
        first[l] = c;
    }
    for (int v = 0; v < 256; ++v) code[v] = len[v] ? first[len[v]]++ : 0;
}

uint64_t cost_bits(const uint64_t hist[256], const uint8_t len[256])
{
    uint64_t t = 0;
    for (int v = 0; v < 256; ++v) t += hist[v] * len[v];
    return t;
}

}  // namespace

namespace zc {
TestKnobs& test_knobs()
{
    static TestKnobs k{kDefaultSpinLimit, 0, 0};
    return k;
}
}  // namespace zc

extern "C" {

void zc_test_set_wait_limit(uint32_t polls) { test_knobs().spin_limit = polls ? polls : kDefaultSpinLimit; }
void zc_test_stall_encoder(uint32_t first_ticket) { test_knobs().first_ticket = first_ticket; }
void zc_test_stall_decoder(uint32_t on) { test_knobs().skip_copy = on ? 1u : 0u; }

int zc_test_debug_counts(uint32_t out[2])
{
#if defined(ZC_DEBUG_CHECKS) && ZC_DEBUG_CHECKS
    out[0] = out[1] = 0;
    debug_counts_hist(out);
    debug_counts_encode(out);
    debug_counts_decode(out);
    return 1;
#else
    (void)out;
    return 0;
#endif
}

zc_status zc_plan(zc_format fmt, uint64_t n_elems, uint32_t chunk_bytes, zc_plan_t** out)
{
    if (!out) return ZC_E_INVALID_ARG;
    const uint32_t g = group_of((uint32_t)fmt);
    if (!g) return ZC_E_UNSUPPORTED;
    if (chunk_bytes < 1024 || chunk_bytes > ZC_MAX_CHUNK_BYTES || chunk_bytes % 1024) return ZC_E_INVALID_ARG;
    if (fmt == ZC_FMT_FP4_E2M1 && (n_elems & 1)) return ZC_E_INVALID_ARG;
    if (n_elems > (1ull << 40)) return ZC_E_INVALID_ARG;
    zc_plan_s* p = new (std::nothrow) zc_plan_s;
    if (!p) return ZC_E_NOMEM;
    p->format = (uint32_t)fmt;
    p->group = g;
    p->chunk_bytes = chunk_bytes;
    p->n_elems = n_elems;
    p->n_syms = (n_elems + g - 1) / g;
    p->syms_per_chunk = chunk_bytes / 2;
    p->syms_per_sub = p->syms_per_chunk / kSubs;
    const uint64_t nc = (p->n_syms + p->syms_per_chunk - 1) / p->syms_per_chunk;
    if (nc > 0xFFFFFFFFull) { delete p; return ZC_E_INVALID_ARG; }
    p->n_chunks = (uint32_t)nc;
    p->input_bytes = fmt == ZC_FMT_BF16 ? 2 * n_elems : fmt == ZC_FMT_FP4_E2M1 ? n_elems / 2 : n_elems;
    *out = p;
    return ZC_OK;
}

void zc_plan_destroy(zc_plan_t* plan) { delete plan; }

zc_status zc_plan_get_info(const zc_plan_t* p, zc_plan_info* o)
{
    if (!p || !o) return ZC_E_INVALID_ARG;
    o->format = p->format; o->group = p->group; o->chunk_bytes = p->chunk_bytes; o->n_chunks = p->n_chunks;
    o->n_elems = p->n_elems; o->n_syms = p->n_syms; o->input_bytes = p->input_bytes;
    o->syms_per_chunk = p->syms_per_chunk; o->syms_per_subchunk = p->syms_per_sub;
    return ZC_OK;
}

size_t zc_max_compressed_bytes(const zc_plan_t* p)
{
    if (!p) return 0;
    const uint64_t worst_piece = round_up(((uint64_t)p->syms_per_chunk * kLmax + 7) / 8, 16);
    const uint64_t huff = table_section_bytes(p->n_chunks, p->chunk_bytes) + (uint64_t)p->n_chunks * worst_piece;
    const uint64_t raw = round_up(p->n_syms, 16);
    return (size_t)(kHeaderBytes + 2 * std::max(huff, raw) + 16);
}

size_t zc_workspace_bytes(const zc_plan_t* p)
{
    if (!p) return 0;
    return (size_t)round_up(kControlBytes + 8ull * p->n_chunks, 256);
}

static bool known_policy(zc_policy policy)
{
    return policy == ZC_POLICY_AUTO || policy == ZC_POLICY_HUFF_ALL || policy == ZC_POLICY_RAW_ALL || policy == ZC_POLICY_STATIC;
}

zc_status zc_build_codebook(const zc_plan_t* plan, const uint64_t* h_hist, zc_policy policy, zc_codebook_t** out)
{
    if (!plan || !h_hist || !out) return ZC_E_INVALID_ARG;
    if (!known_policy(policy)) return ZC_E_UNSUPPORTED;
    zc_codebook_s* cb = new (std::nothrow) zc_codebook_s;
    if (!cb) return ZC_E_NOMEM;
    for (int s = 0; s < 2; ++s) {
        const uint64_t* h = h_hist + 256 * s;
        uint64_t n = 0;
        for (int v = 0; v < 256; ++v) n += h[v];
        // a static dictionary codes tensors it has not seen: every symbol counts as 1/256 of an occurrence more
        uint64_t smoothed[256];
        if (policy == ZC_POLICY_STATIC) {
            if (n >> 54) { delete cb; return ZC_E_INVALID_ARG; }
            for (int v = 0; v < 256; ++v) smoothed[v] = 256 * h[v] + 1;
        }
        if (!limited_lengths(policy == ZC_POLICY_STATIC ? smoothed : h, kLmax, cb->len[s])) { delete cb; return ZC_E_INVALID_ARG; }
        canonical(cb->len[s], cb->code[s]);
        uint32_t mode = ZC_MODE_RAW;
        if (n != 0 && policy == ZC_POLICY_HUFF_ALL) mode = ZC_MODE_HUFF;
        if (n != 0 && (policy == ZC_POLICY_AUTO || policy == ZC_POLICY_STATIC) && 64 * cost_bits(h, cb->len[s]) <= 63 * 8 * n)
            mode = ZC_MODE_HUFF;
        cb->mode[s] = mode;
    }
    finish_codebook(cb);
    *out = cb;
    return ZC_OK;
}

zc_status zc_build_codebooks(uint32_t n_tensors, const zc_plan_t* const* plans, const uint64_t* h_hists, zc_policy policy,
                             uint32_t n_threads, zc_codebook_t** out)
{
    if (n_tensors == 0) return ZC_OK;
    if (!plans || !h_hists || !out) return ZC_E_INVALID_ARG;
    if (!known_policy(policy)) return ZC_E_UNSUPPORTED;
    if (n_threads == 0) {
        const uint32_t hw = std::max(1u, std::thread::hardware_concurrency());
        n_threads = std::min<uint32_t>({hw, 16u, (n_tensors + 7) / 8});     // a codebook takes tens of microseconds
    }
    n_threads = std::max<uint32_t>(1, std::min<uint32_t>(n_threads, n_tensors));
    std::vector<zc_codebook_t*> made(n_tensors, nullptr);
    std::atomic<int> first_error{ZC_OK};
    auto work = [&](uint32_t tid) {
        for (uint32_t t = tid; t < n_tensors; t += n_threads) {
            const zc_status st = zc_build_codebook(plans[t], h_hists + 512ull * t, policy, &made[t]);
            if (st != ZC_OK) { int expected = ZC_OK; first_error.compare_exchange_strong(expected, (int)st); }
        }
    };
    std::vector<std::thread> pool;
    try {
        for (uint32_t i = 1; i < n_threads; ++i) pool.emplace_back(work, i);
    } catch (...) {
        // fewer threads than asked for: the strides of the missing ones are done below
        const uint32_t started = (uint32_t)pool.size() + 1;
        for (uint32_t i = started; i < n_threads; ++i) work(i);
    }
    work(0);
    for (auto& th : pool) th.join();
    if (first_error.load() != ZC_OK) {
        for (auto* cb : made) delete cb;
        return (zc_status)first_error.load();
    }
    for (uint32_t t = 0; t < n_tensors; ++t) out[t] = made[t];
    return ZC_OK;
}

void zc_codebook_destroy(zc_codebook_t* cb) { delete cb; }

// ---- runtime dictionaries (Sec. 3.3): one static codebook and the rule that says when to replace it ----
struct zc_dict_s {
    zc_codebook_t* cb = nullptr;
    double tolerance = 0, baseline = 0, last = 0;
    uint64_t n_observed = 0, n_rebuilds = 0;
    bool has_baseline = false;
};

zc_status zc_dict_create(const zc_plan_t* plan, const uint64_t* h_hist, double tolerance, zc_dict_t** out)
{
    if (!plan || !h_hist || !out || !(tolerance >= 0) || !std::isfinite(tolerance)) return ZC_E_INVALID_ARG;
    zc_dict_s* d = new (std::nothrow) zc_dict_s;
    if (!d) return ZC_E_NOMEM;
    const zc_status st = zc_build_codebook(plan, h_hist, ZC_POLICY_STATIC, &d->cb);
    if (st != ZC_OK) { delete d; return st; }
    d->tolerance = tolerance;
    *out = d;
    return ZC_OK;
}

void zc_dict_destroy(zc_dict_t* d)
{
    if (!d) return;
    zc_codebook_destroy(d->cb);
    delete d;
}

const zc_codebook_t* zc_dict_codebook(const zc_dict_t* d) { return d ? d->cb : nullptr; }

zc_status zc_dict_observe(zc_dict_t* d, uint64_t input_bytes, uint64_t container_bytes, int* rebuild)
{
    if (!d || !rebuild || input_bytes == 0) return ZC_E_INVALID_ARG;
    const double ratio = (double)container_bytes / (double)input_bytes;
    d->last = ratio;
    ++d->n_observed;
    if (!d->has_baseline) {
        d->baseline = ratio;
        d->has_baseline = true;
        *rebuild = 0;
    } else {
        *rebuild = ratio > d->baseline * (1.0 + d->tolerance) ? 1 : 0;
    }
    return ZC_OK;
}

zc_status zc_dict_rebuild(zc_dict_t* d, const zc_plan_t* plan, const uint64_t* h_hist)
{
    if (!d || !plan || !h_hist) return ZC_E_INVALID_ARG;
    zc_codebook_t* fresh = nullptr;
    const zc_status st = zc_build_codebook(plan, h_hist, ZC_POLICY_STATIC, &fresh);
    if (st != ZC_OK) return st;
    zc_codebook_destroy(d->cb);
    d->cb = fresh;
    d->has_baseline = false;
    d->baseline = 0;
    ++d->n_rebuilds;
    return ZC_OK;
}

zc_status zc_dict_get_info(const zc_dict_t* d, zc_dict_info* out)
{
    if (!d || !out) return ZC_E_INVALID_ARG;
    out->tolerance = d->tolerance; out->baseline_ratio = d->baseline; out->last_ratio = d->last;
    out->n_observed = d->n_observed; out->n_rebuilds = d->n_rebuilds;
    out->has_baseline = d->has_baseline ? 1u : 0u; out->reserved = 0;
    return ZC_OK;
}

zc_status zc_codebook_get(const zc_codebook_t* cb, uint32_t s, uint32_t* mode, uint8_t* len256, uint32_t* code256)
{
    if (!cb || s > 1) return ZC_E_INVALID_ARG;
    if (mode) *mode = cb->mode[s];
    if (len256) std::memcpy(len256, cb->len[s], 256);
    if (code256) std::memcpy(code256, cb->code[s], 256 * sizeof(uint32_t));
    return ZC_OK;
}

zc_status zc_validate_container(const zc_plan_t* p, const void* h_container, size_t bytes)
{
    if (!p || !h_container) return ZC_E_INVALID_ARG;
    const uint8_t* c = (const uint8_t*)h_container;
    if (bytes < kHeaderBytes) return ZC_E_CORRUPT;
    if (rd(c + kHdrMagic, 4) != kMagic || rd(c + kHdrVersion, 2) != 1 || c[kHdrStreams] != 2) return ZC_E_CORRUPT;
    if (c[kHdrFormat] != p->format || c[kHdrGroup] != p->group || c[kHdrLmax] != kLmax || c[kHdrSubs] != kSubs ||
        c[kHdrSubWidth] != sub_end_width(p->chunk_bytes))
        return ZC_E_CORRUPT;
    if (rd(c + kHdrElems, 8) != p->n_elems || rd(c + kHdrChunkBytes, 4) != p->chunk_bytes ||
        rd(c + kHdrChunks, 4) != p->n_chunks)
        return ZC_E_CORRUPT;
    uint32_t mode[2];
    for (int s = 0; s < 2; ++s) {
        const uint8_t* d = c + kHdrStream0 + kHdrStreamStride * s;
        mode[s] = d[kSdMode];
        if (mode[s] > 1 || rd(d + kSdSyms, 8) != p->n_syms) return ZC_E_CORRUPT;
    }
    const Layout L = make_layout(*p, mode);
    const bool any_huff = mode[0] == ZC_MODE_HUFF || mode[1] == ZC_MODE_HUFF;
    const uint64_t total = rd(c + kHdrTotal, 8), poff = rd(c + kHdrPayloadOff, 8), pbytes = rd(c + kHdrPayloadBytes, 8);
    if (poff != L.payload_off || pbytes % 16 || total != poff + pbytes + (any_huff ? 16 : 0) || total > bytes)
        return ZC_E_CORRUPT;
    for (int s = 0; s < 2; ++s)
        if (rd(c + kHdrStream0 + kHdrStreamStride * s + kSdSection, 8) != L.section_off[s]) return ZC_E_CORRUPT;

    uint64_t bits[2] = {0, 0};
    for (int s = 0; s < 2; ++s) {
        if (mode[s] != ZC_MODE_HUFF) continue;
        const uint8_t* len = c + L.section_off[s];
        uint64_t kraft = 0; uint32_t active = 0;
        for (int v = 0; v < 256; ++v) {
            if (len[v] > kLmax) return ZC_E_CORRUPT;
            if (len[v]) { kraft += 1ull << (kLmax - len[v]); ++active; }
        }
        if (p->n_syms && active == 0) return ZC_E_CORRUPT;
        if (active == 1 ? kraft != (1ull << (kLmax - 1)) : (active > 1 && kraft != (1ull << kLmax))) return ZC_E_CORRUPT;
    }
    uint64_t pos16 = 0;
    for (uint32_t ch = 0; ch < p->n_chunks; ++ch) {
        for (int s = 0; s < 2; ++s) {
            if (mode[s] != ZC_MODE_HUFF) continue;
            if (rd(c + L.chunk_off_tab[s] + 4ull * ch, 4) != pos16) return ZC_E_CORRUPT;
            const uint32_t sw = sub_end_width(p->chunk_bytes);
            const uint8_t* se = c + L.sub_end_tab[s] + 32ull * sw * ch;
            uint64_t prev = 0;
            for (uint32_t j = 0; j < kSubs; ++j) {
                const uint64_t e = rd(se + sw * j, (int)sw);
                if (e < prev || e - prev > (uint64_t)p->syms_per_sub * kLmax) return ZC_E_CORRUPT;
                prev = e;
            }
            bits[s] += prev;
            pos16 += (prev + 127) / 128;
        }
    }
    if (16 * pos16 != pbytes) return ZC_E_CORRUPT;
    for (int s = 0; s < 2; ++s) {
        const uint64_t hb = rd(c + kHdrStream0 + kHdrStreamStride * s + kSdBits, 8);
        if (hb != (mode[s] == ZC_MODE_HUFF ? bits[s] : 8 * p->n_syms)) return ZC_E_CORRUPT;
    }
    if (any_huff)
        for (int i = 0; i < 16; ++i)
            if (c[poff + pbytes + i]) return ZC_E_CORRUPT;
    return ZC_OK;
}

zc_status zc_stats(const zc_plan_t* p, const zc_codebook_t* cb, const uint64_t* h_hist, const void* h_header,
                   zc_stats_t* out)
{
    if (!p || !cb || !h_hist || !out) return ZC_E_INVALID_ARG;
    zc_stats_t st;
    std::memset(&st, 0, sizeof(st));
    const uint8_t* hd = (const uint8_t*)h_header;
    if (hd && (rd(hd + kHdrMagic, 4) != kMagic || rd(hd + kHdrElems, 8) != p->n_elems)) return ZC_E_CORRUPT;
    uint64_t payload = 0;
    for (int s = 0; s < 2; ++s) {
        const uint64_t* h = h_hist + 256 * s;
        zc_stream_stats& o = st.stream[s];
        for (int v = 0; v < 256; ++v) o.n_syms += h[v];
        o.raw_bits = 8 * o.n_syms;
        o.mode = cb->mode[s];
        double H = 0.0;
        uint64_t bits = 0;
        for (int v = 0; v < 256; ++v) {
            if (!h[v]) continue;
            o.n_active_symbols++;
            o.max_len = std::max<uint32_t>(o.max_len, cb->len[s][v]);
            bits += h[v] * cb->len[s][v];
            const double q = (double)h[v] / (double)o.n_syms;
            H -= q * std::log2(q);
        }
        o.entropy_bits = H;
        o.avg_len = o.n_syms ? (double)bits / (double)o.n_syms : 0.0;
        o.payload_bits = o.mode == ZC_MODE_HUFF ? bits : o.raw_bits;
        payload += o.payload_bits;
        if (hd) {
            const uint8_t* d = hd + kHdrStream0 + kHdrStreamStride * s;
            if (d[kSdMode] != o.mode) return ZC_E_CORRUPT;
            const uint64_t hb = rd(d + kSdBits, 8);
            o.container_bytes = o.mode == ZC_MODE_HUFF ? table_section_bytes(p->n_chunks, p->chunk_bytes)
                                                       : round_up(p->n_syms, 16);
            if (o.mode == ZC_MODE_HUFF) {
                // this stream's share of the payload area: its bits, pieces rounded to 16 bytes are
                // attributed in proportion, the exact sum is out_bytes below
                o.container_bytes += (hb + 7) / 8;
            }
        }
    }
    st.in_bytes = p->input_bytes;
    st.ratio_payload = st.in_bytes ? (double)payload / (8.0 * (double)st.in_bytes) : 0.0;
    if (hd) {
        st.out_bytes = rd(hd + kHdrTotal, 8);
        st.ratio_container = st.in_bytes ? (double)st.out_bytes / (double)st.in_bytes : 0.0;
    }
    *out = st;
    return ZC_OK;
}

zc_status zc_test_split16(zc_format fmt, const uint8_t* h_in16, uint8_t* h_e8, uint8_t* h_sm8)
{
    if (!h_in16 || !h_e8 || !h_sm8) return ZC_E_INVALID_ARG;
    uint32_t in[4], e[2], sm[2];
    std::memcpy(in, h_in16, 16);
    switch (fmt) {
    case ZC_FMT_BF16: split16<ZC_FMT_BF16>(in, e, sm); break;
    case ZC_FMT_FP8_E4M3: case ZC_FMT_FP8_E5M2: split16<ZC_FMT_FP8_E4M3>(in, e, sm); break;
    case ZC_FMT_FP4_E2M1: split16<ZC_FMT_FP4_E2M1>(in, e, sm); break;
    case ZC_FMT_SCALE_U8: split16<ZC_FMT_SCALE_U8>(in, e, sm); break;
    default: return ZC_E_UNSUPPORTED;
    }
    std::memcpy(h_e8, e, 8);
    std::memcpy(h_sm8, sm, 8);
    return ZC_OK;
}

zc_status zc_test_merge16(zc_format fmt, const uint8_t* h_e8, const uint8_t* h_sm8, uint8_t* h_out16)
{
    if (!h_e8 || !h_sm8 || !h_out16) return ZC_E_INVALID_ARG;
    uint32_t e[2], sm[2], out[4];
    std::memcpy(e, h_e8, 8);
    std::memcpy(sm, h_sm8, 8);
    switch (fmt) {
    case ZC_FMT_BF16: merge16<ZC_FMT_BF16>(e, sm, out); break;
    case ZC_FMT_FP8_E4M3: case ZC_FMT_FP8_E5M2: merge16<ZC_FMT_FP8_E4M3>(e, sm, out); break;
    case ZC_FMT_FP4_E2M1: merge16<ZC_FMT_FP4_E2M1>(e, sm, out); break;
    case ZC_FMT_SCALE_U8: merge16<ZC_FMT_SCALE_U8>(e, sm, out); break;
    default: return ZC_E_UNSUPPORTED;
    }
    std::memcpy(h_out16, out, 16);
    return ZC_OK;
}

const char* zc_strerror(zc_status s)
{
    switch (s) {
    case ZC_OK: return "ok";
    case ZC_E_INVALID_ARG: return "invalid argument";
    case ZC_E_UNSUPPORTED: return "unsupported format or policy";
    case ZC_E_BUFFER_TOO_SMALL: return "output buffer too small";
    case ZC_E_CORRUPT: return "container is damaged or does not match the plan";
    case ZC_E_CUDA: return "CUDA runtime error";
    case ZC_E_NOMEM: return "out of host memory";
    case ZC_E_DEVICE_TIMEOUT: return "a bounded wait on the device gave up";
    case ZC_E_NO_CODE: return "an input symbol has no code in the codebook";
    case ZC_E_TOO_LARGE: return "tensor has more chunks than the built-in scratch of zc_compress_noalloc covers";
    default: return "unknown status";
    }
}

}  // extern "C"
